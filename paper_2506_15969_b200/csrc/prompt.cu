// Causal attention over the prompt with recurrence tracking from the first prompt token.
//
// For every cache unit and every prompt row j (Appendix A, Eq. (attn), with a causal mask):
//   s_g[j][i] = q_{j,g} . k_i / sqrt(D),  i <= j;   p_g[j] = softmax_i(s_g[j]);   out_{j,g} = sum_i p_g[j][i] v_i
//   pbar[j][i] = mean_g p_g[j][i]
// and, in row order (Section 4 "Recurrence Interval Tracking", Eq. (1), Algorithm 1's loop),
//   pbar[j][i] >= alpha  =>  MRI[i] = max(MRI[i], time_j - TS[i]);  TS[i] = time_j,   time_j = j - (P - 1).
//
// This is the one dense contraction of the path, so it runs on the fifth-generation tensor cores:
// tcgen05.mma with operands in shared memory (TMA tiles, 128-byte swizzle) or tensor memory and
// accumulators in tensor memory.  One block owns a unit and walks its query tiles in row order; a query
// tile is 128 rows = (128 / GP) prompt positions x GP query-head slots (GP = 4 or 8, the group size
// rounded up), so the heads that share the K / V tile sit in neighbouring lanes.  Every query tile
// makes two passes over its key tiles (128 keys each):
//   pass A: S = Q K^T, row maximum and sum of exponentials  ->  exact log-sum-exp per row;
//   pass B: S = Q K^T again, p = exp2(s - lse) (already normalised) written back over S in tensor
//           memory as two bf16 terms (hi + lo), O += P V with P as the tensor-memory operand (no
//           rescaling ever, no shared-memory round trip), pbar by a butterfly sum over the GP lanes of
//           a position, threshold test, activation bits per key column; after the tile one thread per
//           key column applies Eq. (1) for the tile's positions in ascending order.
// Key columns are owned by a fixed thread for the whole unit and query tiles are visited in ascending
// order, so every token sees its activations in row order.
//
// Pipeline: S is double-buffered in tensor memory, so the tensor core computes the logits of key tile
// kb + 1 (and, in pass B, O += P V of tile kb - 1) while the softmax warps work on tile kb; K tiles come
// through a three-stage ring, V tiles through a two-stage ring, and the next query tile's Q is fetched
// while the current one is worked on.  MMAs issued by one thread execute in issue order, which is what
// orders "O += P V of tile kb" before "S of tile kb + 2" on the same tensor-memory columns.
//
// Warp roles: warps 0-15 softmax / tracking / epilogue (thread = accumulator row = TMEM lane; the four
// warps that share a lane quarter take 32 of a tile's columns each), warp 16 TMA producer,
// warp 17 MMA issuer.  All mbarrier waits are bounded.
#include <cuda.h>

#include "internal.h"

namespace lzk {

namespace {

constexpr int kTile = 128;                         // rows of a query tile, keys of a key tile
constexpr int kBoxBytes = kTile * 128;             // one TMA box: 128 rows x 64 bf16 (16 KiB)
constexpr int kOperandBytes = 2 * kBoxBytes;       // a 128 x 128 bf16 operand tile: two boxes (32 KiB)
constexpr int kKStages = 3, kVStages = 2;
constexpr int kSoftmaxWarps = 16;                  // four per TMEM lane quarter: each takes 32 of a tile's 128 columns
constexpr int kSoftmaxThreads = 32 * kSoftmaxWarps;
constexpr int kPromptThreads = kSoftmaxThreads + 64;

// shared-memory map (the base is 1024-byte aligned: the swizzle atoms need it)
constexpr int kOffQ = 0;                                            // two query tiles
constexpr int kOffK = kOffQ + 2 * kOperandBytes;
constexpr int kOffV = kOffK + kKStages * kOperandBytes;
constexpr int kOffMisc = kOffV + kVStages * kOperandBytes;
constexpr int kMiscBytes = 2048;
constexpr int kPromptSmem = kOffMisc + kMiscBytes;                  // 226 KiB of the 227 KiB a block may have

// tensor-memory columns: S / P double buffer, O, and a few spare columns for the row statistics
constexpr uint32_t kColS = 0, kColO = 256, kColStats = 384, kTmemCols = 512;

struct Bars {                                       // mbarriers
    uint64_t q_full[2], out_ready[2];               // out_ready: the tile's output sits in its Q slot
    uint64_t k_full[kKStages], k_empty[kKStages];
    uint64_t v_full[kVStages], v_empty[kVStages];
    uint64_t s_full[2], s_empty[2];
    uint64_t p_full[2];
    uint64_t o_full, o_empty;
    uint64_t drain;
};

struct PromptParams {
    int units, group, P, capacity;
    float scale_log2, inv_group, alpha;
    int2* tsm;                                      // (TS, MRI) per token
    float* pbar;
    int32_t* status;
    float* dump;                                    // optional: [dump_count][P][P] probabilities per prompt row
    int dump_begin, dump_count;
    unsigned long long wait_limit_ns;
    int stop_after_tiles;                           // diagnostics: the producer stops after this many K tiles (-1: off)
};

// ---- PTX wrappers used only here ------------------------------------------------------------------
__device__ __forceinline__ void tma_load_3d(void* smem_dst, const CUtensorMap* map, int x, int y, int z, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
            smem_u32(smem_dst)),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
        : "memory");
}

__device__ __forceinline__ void tma_load_4d(void* smem_dst, const CUtensorMap* map, int x, int y, int z, int w,
                                            uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];" ::"r"(
            smem_u32(smem_dst)),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(w), "r"(smem_u32(bar))
        : "memory");
}

// Tile store shared -> global through a tensor map (rows outside the tensor are dropped).
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, int x, int y, int z, int w, const void* smem_src) {
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3, %4}], [%5];" ::"l"(
                     reinterpret_cast<uint64_t>(map)),
                 "r"(x), "r"(y), "r"(z), "r"(w), "r"(smem_u32(smem_src))
                 : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void umma_commit(uint64_t* bar) {     // arrives once the MMAs issued so far are done
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

// D[tmem] (+)= A[smem] * B[smem], 128 x 128 x 16, bf16 in, fp32 accumulate.
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
        "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}

// The same with A in tensor memory (row i in lane i, two bf16 per 32-bit column, 8 columns per instruction).
__device__ __forceinline__ void umma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t desc_b, uint32_t idesc,
                                             uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(tmem_d),
        "r"(tmem_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
        "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]),
        "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
        : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7]), "=f"(v[8]),
          "=f"(v[9]), "=f"(v[10]), "=f"(v[11]), "=f"(v[12]), "=f"(v[13]), "=f"(v[14]), "=f"(v[15]), "=f"(v[16]),
          "=f"(v[17]), "=f"(v[18]), "=f"(v[19]), "=f"(v[20]), "=f"(v[21]), "=f"(v[22]), "=f"(v[23]), "=f"(v[24]),
          "=f"(v[25]), "=f"(v[26]), "=f"(v[27]), "=f"(v[28]), "=f"(v[29]), "=f"(v[30]), "=f"(v[31])
        : "r"(taddr)
        : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle, rows (or key rows) of 128 bytes, eight of them per
// 1024-byte swizzle atom.  K-major operands: the leading offset is unused (1), the stride offset steps
// between groups of eight rows.  MN-major operands (V: keys x dims with dims contiguous): the leading
// offset steps between the two 64-element column blocks, the stride offset between groups of eight keys.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t leading_bytes, uint32_t stride_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFF) >> 4);
    d |= (uint64_t)(leading_bytes >> 4) << 16;
    d |= (uint64_t)(stride_bytes >> 4) << 32;
    d |= (uint64_t)1 << 46;                        // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                        // 128-byte swizzle
    return d;
}

// Instruction descriptor: fp32 accumulator, bf16 A and B, M = 128, N = 128; b_mn_major = B is MN-major.
__host__ __device__ constexpr uint32_t instr_desc(bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
}

// Has the phase with this parity completed?  Never suspends the thread (try_wait may, for a while).
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Sleep until the phase completes or about `ns` nanoseconds have passed, whichever is first: a wait that
// leaves the issue slots to the other warps of the scheduler, unlike a polling loop.
__device__ __forceinline__ void mbar_nap(uint64_t* bar, uint32_t parity, uint32_t ns) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%0], %1, %2;\n\t}" ::"r"(smem_u32(bar)),
        "r"(parity), "r"(ns)
        : "memory");
}

// Bounded wait on an mbarrier phase; on time-out the abort flag and the device status word are set
// and no later wait blocks.
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                         unsigned long long limit_ns, bool honour_abort = true) {
    if (mbar_try_wait(bar, parity)) return true;
    if (honour_abort && *abort_flag) return false;
    uint32_t spins = 0;
    uint64_t t_start = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 0x3F) == 0) {
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

// Two fp32 lanes per instruction (packed .f32x2 arithmetic) and the three-input maximum: the softmax warps
// are bound by the number of instructions they issue per logit, not by any one pipe.  Each lane rounds
// exactly like the scalar instruction, so results do not depend on which form is used.
__device__ __forceinline__ uint64_t pack2(float a, float b) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t r, float& a, float& b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(r)); }
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// One use of a barrier pair in a ring: which stage and which parity a counter of uses maps to.
struct Ring {
    uint32_t count = 0;
    __device__ __forceinline__ uint32_t stage(uint32_t n) const { return count % n; }
    __device__ __forceinline__ uint32_t parity(uint32_t n) const { return (count / n) & 1u; }
};

template <int GP>
__global__ void __launch_bounds__(kPromptThreads, 1)
prompt_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
              const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_out,
              const PromptParams p) {
    constexpr int TQ = kTile / GP;                  // prompt positions per query tile
    extern __shared__ __align__(1024) uint8_t smem[];
    Bars* bars = reinterpret_cast<Bars*>(smem + kOffMisc);
    uint32_t* act = reinterpret_cast<uint32_t*>(smem + kOffMisc + 512);          // [2][128] activation bits per key column
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kOffMisc + 512 + 1024);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int P = p.P, G = p.group;

    if (threadIdx.x == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(&bars->q_full[i], 1);
            mbar_init(&bars->out_ready[i], kSoftmaxWarps);
            mbar_init(&bars->s_full[i], 1);
            mbar_init(&bars->s_empty[i], kSoftmaxWarps);
            mbar_init(&bars->p_full[i], kSoftmaxWarps);
        }
        for (int i = 0; i < kKStages; ++i) {
            mbar_init(&bars->k_full[i], 1);
            mbar_init(&bars->k_empty[i], 1);
        }
        for (int i = 0; i < kVStages; ++i) {
            mbar_init(&bars->v_full[i], 1);
            mbar_init(&bars->v_empty[i], 1);
        }
        mbar_init(&bars->o_full, 1);
        mbar_init(&bars->o_empty, kSoftmaxWarps);
        mbar_init(&bars->drain, 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    for (int i = threadIdx.x; i < 256; i += kPromptThreads) act[i] = 0u;
    if (warp == 0) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish_alloc_permit();
    }
    tmem_fence_before_sync();
    __syncthreads();
    tmem_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    const unsigned long long limit = p.wait_limit_ns;

    const int n_qt = (P + TQ - 1) / TQ;
    // key tiles a query tile needs: all keys up to its last position
    auto key_tiles = [&](int qt) { return (min(P, (qt + 1) * TQ) - 1) / kTile + 1; };

    if (warp == kSoftmaxWarps) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            Ring kr, vr, qr;                        // uses of the K ring, the V ring and the two Q slots
            bool ok = true;
            int slot_u[2] = {0, 0}, slot_qt[2] = {0, 0};
            auto store_out = [&](uint32_t qs) {    // the output tile in slot qs -> out[positions][unit][heads][128]
                const uint8_t* o_s = smem + kOffQ + qs * kOperandBytes;
                tma_store_4d(&map_out, 0, 0, slot_u[qs], slot_qt[qs] * TQ, o_s);
                tma_store_4d(&map_out, 64, 0, slot_u[qs], slot_qt[qs] * TQ, o_s + kBoxBytes);
                tma_store_commit();
                tma_store_wait_read();              // the slot may be overwritten from here on
            };
            for (int u = blockIdx.x; u < p.units && ok; u += gridDim.x) {
                for (int qt = 0; qt < n_qt && ok; ++qt) {
                    {
                        // The slot's previous query tile left its attention output there (the softmax warps
                        // wrote it once the tile's MMAs were done): send it off, then refill the slot.
                        const uint32_t qs = qr.stage(2);
                        if (qr.count >= 2) {
                            ok = wait_bar(&bars->out_ready[qs], qr.parity(2) ^ 1u, abort_flag, p.status, limit);
                            if (!ok) break;
                            store_out(qs);
                        }
                        slot_u[qs] = u;
                        slot_qt[qs] = qt;
                        uint8_t* q_s = smem + kOffQ + qs * kOperandBytes;
                        mbar_arrive_expect_tx(&bars->q_full[qs], kOperandBytes);
                        tma_load_4d(q_s, &map_q, 0, 0, u, qt * TQ, &bars->q_full[qs]);
                        tma_load_4d(q_s + kBoxBytes, &map_q, 64, 0, u, qt * TQ, &bars->q_full[qs]);
                        ++qr.count;
                    }
                    const int nkb = key_tiles(qt);
                    for (int pass = 0; pass < 2 && ok; ++pass) {
                        for (int kb = 0; kb < nkb; ++kb) {
                            const uint32_t ks = kr.stage(kKStages);
                            // diagnostics: no copy beyond the first stop_after_tiles K tiles -- the other roles wait
                            // for a tile that never comes, give up after the wait limit and flag the status word
                            ok = p.stop_after_tiles < 0 || (int)kr.count < p.stop_after_tiles;
                            if (!ok) break;
                            ok = wait_bar(&bars->k_empty[ks], kr.parity(kKStages) ^ 1u, abort_flag, p.status, limit);
                            if (!ok) break;
                            uint8_t* k_s = smem + kOffK + ks * kOperandBytes;
                            mbar_arrive_expect_tx(&bars->k_full[ks], kOperandBytes);
                            tma_load_3d(k_s, &map_k, 0, kb * kTile, u, &bars->k_full[ks]);
                            tma_load_3d(k_s + kBoxBytes, &map_k, 64, kb * kTile, u, &bars->k_full[ks]);
                            ++kr.count;
                            if (pass == 1) {
                                const uint32_t vs = vr.stage(kVStages);
                                ok = wait_bar(&bars->v_empty[vs], vr.parity(kVStages) ^ 1u, abort_flag, p.status, limit);
                                if (!ok) break;
                                uint8_t* v_s = smem + kOffV + vs * kOperandBytes;
                                mbar_arrive_expect_tx(&bars->v_full[vs], kOperandBytes);
                                tma_load_3d(v_s, &map_v, 0, kb * kTile, u, &bars->v_full[vs]);
                                tma_load_3d(v_s + kBoxBytes, &map_v, 64, kb * kTile, u, &bars->v_full[vs]);
                                ++vr.count;
                            }
                        }
                    }
                }
            }
            if (ok) {
                // the outputs of the last two query tiles
                const uint32_t pending = qr.count < 2 ? qr.count : 2;
                for (uint32_t k = qr.count - pending; k < qr.count && ok; ++k) {
                    ok = wait_bar(&bars->out_ready[k & 1u], (k >> 1) & 1u, abort_flag, p.status, limit);
                    if (ok) store_out(k & 1u);
                }
            }
            tma_store_wait_all();
            if (!ok) {
                // Aborted: let the copies already issued land before the block exits (the last uses of
                // every stage may still be in flight).
                auto drain = [&](uint64_t* full, const Ring& r, uint32_t n) {
                    const uint32_t last = r.count < n ? r.count : n;
                    for (uint32_t k = r.count - last; k < r.count; ++k)
                        wait_bar(&full[k % n], (k / n) & 1u, abort_flag, p.status, limit, false);
                };
                drain(bars->k_full, kr, kKStages);
                drain(bars->v_full, vr, kVStages);
                drain(bars->q_full, qr, 2);
            }
        }
    } else if (warp == kSoftmaxWarps + 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            // Two cursors walk the same sequence of (unit, query tile) pairs.  The S cursor issues the logits
            // products -- per query tile one per key tile for pass A, then one per key tile for pass B; job j goes
            // to S buffer j % 2 -- and the O cursor issues O += P V behind the softmax warps.  The S cursor may be
            // up to one job past the O cursor's job: the job after that would overwrite the P the O cursor is
            // about to read.  Its run-ahead crosses query tile and unit boundaries, so the first logits of the next
            // query tile are computed while the softmax warps still work on the last key tile of this one.  The
            // thread polls both cursors and issues whichever has everything it needs; it never blocks on one
            // while the other could go (a late Q or K tile must not hold back the product that completes O).
            Ring kr, vr, sq, sb;                    // K and V ring uses, query tiles begun by the S cursor, S jobs issued
            uint32_t p_cnt0 = 0, p_cnt1 = 0, o_uses = 0;
            const uint32_t idesc_s = instr_desc(false), idesc_o = instr_desc(true);
            const uint32_t tmem_o = tmem_base + kColO;
            int s_u = blockIdx.x, s_qt = 0, s_pass = 0, s_kb = 0, s_nkb = key_tiles(0);
            bool s_more = s_u < p.units;
            int o_u = blockIdx.x, o_qt = 0, o_kb = 0, o_nkb = key_tiles(0);
            bool o_more = o_u < p.units;
            uint32_t o_job = (uint32_t)o_nkb;       // the pass B job whose P the O cursor's next product reads
            uint32_t q_addr = 0;
            uint32_t spins = 0;
            uint64_t t_start = 0;
            while (o_more) {
                bool issued = false;
                uint64_t* nap_bar = nullptr;        // a barrier whose phase one of the cursors is waiting for
                uint32_t nap_parity = 0;
                {
                    // ---- O += P V for key tile o_kb, once P is there (and V, and for the first tile the old O is out)
                    const uint32_t buf = o_job & 1u, vs = vr.stage(kVStages);
                    const uint32_t p_par = (buf ? p_cnt1 : p_cnt0) & 1u;
                    if (!mbar_test_wait(&bars->p_full[buf], p_par)) {
                        nap_bar = &bars->p_full[buf];
                        nap_parity = p_par;
                    } else if (!mbar_test_wait(&bars->v_full[vs], vr.parity(kVStages))) {
                        nap_bar = &bars->v_full[vs];
                        nap_parity = vr.parity(kVStages);
                    } else if (o_kb == 0 && !mbar_test_wait(&bars->o_empty, (o_uses & 1u) ^ 1u)) {
                        nap_bar = &bars->o_empty;
                        nap_parity = (o_uses & 1u) ^ 1u;
                    } else {
                        tmem_fence_after_sync();
                        const uint32_t v_addr = smem_u32(smem + kOffV + vs * kOperandBytes);
                        const uint32_t p_col = tmem_base + kColS + buf * 128;
#pragma unroll
                        for (int s8 = 0; s8 < 8; ++s8) {            // 16 keys per instruction; P = hi + lo, two products
                            const uint64_t v_desc = smem_desc(v_addr + s8 * 2048, kBoxBytes, 1024);
                            const uint32_t a_col = p_col + (s8 >> 1) * 32 + (s8 & 1) * 8;
                            umma_bf16_ts(tmem_o, a_col, v_desc, idesc_o, (o_kb > 0 || s8 > 0));
                            umma_bf16_ts(tmem_o, a_col + 16, v_desc, idesc_o, 1u);
                        }
                        umma_commit(&bars->v_empty[vs]);
                        ++vr.count;
                        if (buf) ++p_cnt1; else ++p_cnt0;
                        ++o_job;
                        if (++o_kb == o_nkb) {
                            umma_commit(&bars->o_full);             // the query tile's output is complete
                            ++o_uses;
                            o_kb = 0;
                            if (++o_qt == n_qt) {
                                o_qt = 0;
                                o_u += gridDim.x;
                                o_more = o_u < p.units;
                            }
                            o_nkb = key_tiles(o_qt);
                            o_job += (uint32_t)o_nkb;               // past the next query tile's pass A jobs
                        }
                        issued = true;
                    }
                }
                if (!issued && s_more && sb.count <= o_job + 1) {
                    // ---- S[buffer] = Q K^T for the S cursor's job.  The buffer's previous job (two back) is behind:
                    // the softmax warps have let go of it and, where they left P there, the product that reads
                    // it was issued above, earlier.
                    const uint32_t ks = kr.stage(kKStages), buf = sb.stage(2), qs = sq.stage(2);
                    const bool new_tile = s_pass == 0 && s_kb == 0;
                    // (what the logits wait for comes sooner than P wherever both are missing)
                    if (!mbar_test_wait(&bars->s_empty[buf], sb.parity(2) ^ 1u)) {
                        nap_bar = &bars->s_empty[buf];
                        nap_parity = sb.parity(2) ^ 1u;
                    } else if (!mbar_test_wait(&bars->k_full[ks], kr.parity(kKStages))) {
                        nap_bar = &bars->k_full[ks];
                        nap_parity = kr.parity(kKStages);
                    } else if (new_tile && !mbar_test_wait(&bars->q_full[qs], sq.parity(2))) {
                        nap_bar = &bars->q_full[qs];
                        nap_parity = sq.parity(2);
                    } else {
                        if (new_tile) q_addr = smem_u32(smem + kOffQ + qs * kOperandBytes);
                        tmem_fence_after_sync();
                        const uint32_t k_addr = smem_u32(smem + kOffK + ks * kOperandBytes);
#pragma unroll
                        for (int s8 = 0; s8 < 8; ++s8) {    // 16 head dimensions per instruction: 32 bytes inside a box row
                            const uint32_t off = (s8 >> 2) * kBoxBytes + (s8 & 3) * 32;
                            umma_bf16(tmem_base + kColS + buf * 128, smem_desc(q_addr + off, 16, 1024),
                                      smem_desc(k_addr + off, 16, 1024), idesc_s, s8 > 0);
                        }
                        umma_commit(&bars->s_full[buf]);
                        umma_commit(&bars->k_empty[ks]);
                        ++kr.count;
                        ++sb.count;
                        if (++s_kb == s_nkb) {
                            s_kb = 0;
                            if (++s_pass == 2) {
                                s_pass = 0;
                                ++sq.count;
                                if (++s_qt == n_qt) {
                                    s_qt = 0;
                                    s_u += gridDim.x;
                                    s_more = s_u < p.units;
                                }
                                s_nkb = key_tiles(s_qt);
                            }
                        }
                        issued = true;
                    }
                }
                if (issued) {
                    spins = 0;
                    t_start = 0;
                    continue;
                }
                mbar_nap(nap_bar, nap_parity, 400);
                if ((++spins & 0x3F) == 0) {
                    // nothing could be issued for a while: give up on another role's abort or on the time limit
                    if (*abort_flag) break;
                    const uint64_t now = global_timer_ns();
                    if (t_start == 0) {
                        t_start = now;
                    } else if (now - t_start > limit) {
                        *abort_flag = 1;
                        atomicOr(p.status, kStatusWaitTimeout);
                        break;
                    }
                }
            }
            // every MMA issued by this thread is complete before tensor memory goes back
            umma_commit(&bars->drain);
            wait_bar(&bars->drain, 0, abort_flag, p.status, limit, false);
        }
    } else {
        // ------------------------------------------------------------------ softmax, tracking, epilogue
        // Warps w, w + 4, w + 8, w + 12 share TMEM lanes 32 (w % 4) ..: thread = accumulator row, and the four
        // warps of a row take 32 columns of every tile each (sixteen warps, four per scheduler: the work
        // is a long chain of exponentials, conversions and shuffles, and needs the warps to hide it).
        const int row = threadIdx.x & 127;          // accumulator row = TMEM lane
        const int c = threadIdx.x >> 7;             // which 32 columns of a tile (and of the output)
        const int jj = row / GP, g = row % GP;
        const bool head_on = g < G;
        const uint32_t tmem_row = tmem_base + ((uint32_t)(32 * (warp & 3)) << 16);
        const uint32_t tmem_ml = tmem_row + kColStats;      // the two halves of a row exchange (maximum, sum) here
        // A wait that gives up makes this thread "dead": it keeps walking the same loops, so that every
        // barrier below still gets all its threads, but it waits for nothing any more (once the abort flag
        // is up no wait blocks) and what it computes no longer means anything.
        Ring sb, qr;
        uint32_t o_uses = 0, tiles = 0;
        bool dead = false;
        auto wait_on = [&](uint64_t* bar, uint32_t parity) {
            if (!dead) dead = !wait_bar(bar, parity, abort_flag, p.status, limit);
        };
        // ---- a query tile's attention output: bf16 into the tile's own Q slot (its MMAs are done), in the swizzled
        // layout a TMA store expects; the producer warp sends it off before it refills the slot.
        auto write_output = [&](uint32_t slot) {
            wait_on(&bars->o_full, o_uses & 1u);
            tmem_fence_after_sync();
            {
                float x[32];
                tmem_ld32(tmem_row + kColO + c * 32, x);
                tmem_wait_ld();
                tmem_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars->o_empty);     // the accumulator is in registers
                uint8_t* orow = smem + kOffQ + slot * kOperandBytes + (c >> 1) * kBoxBytes + row * 128;
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    uint4 w;
                    w.x = pack_bf16(x[8 * ch + 0], x[8 * ch + 1]);
                    w.y = pack_bf16(x[8 * ch + 2], x[8 * ch + 3]);
                    w.z = pack_bf16(x[8 * ch + 4], x[8 * ch + 5]);
                    w.w = pack_bf16(x[8 * ch + 6], x[8 * ch + 7]);
                    const int chunk = (c & 1) * 4 + ch;
                    *reinterpret_cast<uint4*>(orow + ((chunk ^ (row & 7)) << 4)) = w;
                }
            }
            fence_proxy_async();                // the store reads shared memory through the async proxy
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->out_ready[slot]);
            ++o_uses;
        };
        for (int u = blockIdx.x; u < p.units; u += gridDim.x) {
            const size_t srow = (size_t)u * p.capacity;
            const bool dumping = p.dump != nullptr && u >= p.dump_begin && u < p.dump_begin + p.dump_count;
            for (int qt = 0; qt < n_qt; ++qt, ++qr.count) {
                const int pos = qt * TQ + jj;
                const int warp_last_pos = qt * TQ + (32 * (warp & 3)) / GP + 32 / GP - 1;      // of this warp's 32 rows
                const int nkb = key_tiles(qt);
                // ---- pass A: exact log-sum-exp of the row (log2 domain) ----
                float m = -INFINITY, l = 0.f;
                for (int kb = 0; kb < nkb; ++kb, ++sb.count) {
                    const uint32_t buf = sb.stage(2);
                    wait_on(&bars->s_full[buf], sb.parity(2));
                    tmem_fence_after_sync();
                    // On the diagonal tile a whole chunk of 32 keys can lie beyond every position of this warp's rows:
                    // nothing of it counts (with short prompts that is a third of all the chunks).
                    if (kb * kTile + c * 32 <= warp_last_pos) {
                        float x[32];
                        tmem_ld32(tmem_row + kColS + buf * 128 + c * 32, x);
                        tmem_wait_ld();
                        tmem_fence_before_sync();   // the logits are in registers: the buffer can be refilled
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&bars->s_empty[buf]);
                        const int key0 = kb * kTile + c * 32;
                        if (key0 + 31 > pos) {      // only the tile on the diagonal has keys beyond the row's position
#pragma unroll
                            for (int i = 0; i < 32; ++i) x[i] = key0 + i <= pos ? x[i] : -INFINITY;
                        }
                        float c0 = fmax3(x[0], x[1], x[2]), c1 = fmax3(x[3], x[4], x[5]);
#pragma unroll
                        for (int i = 6; i < 30; i += 4) {
                            c0 = fmax3(c0, x[i], x[i + 1]);
                            c1 = fmax3(c1, x[i + 2], x[i + 3]);
                        }
                        const float cmax = fmax3(c0, c1, fmaxf(x[30], x[31])) * p.scale_log2;      // the scale is positive
                        if (cmax > m) {
                            l *= fast_exp2(m - cmax);     // m = -inf only while l = 0
                            m = cmax;
                        }
                        if (m > -INFINITY) {
                            const uint64_t scale2 = pack2(p.scale_log2, p.scale_log2), minus_m = pack2(-m, -m);
                            uint64_t l01 = pack2(0.f, 0.f), l23 = l01;
#pragma unroll
                            for (int i = 0; i < 32; i += 4) {
                                float e0, e1, e2, e3;
                                unpack2(fma2(pack2(x[i], x[i + 1]), scale2, minus_m), e0, e1);
                                unpack2(fma2(pack2(x[i + 2], x[i + 3]), scale2, minus_m), e2, e3);
                                l01 = add2(l01, pack2(fast_exp2(e0), fast_exp2(e1)));
                                l23 = add2(l23, pack2(fast_exp2(e2), fast_exp2(e3)));
                            }
                            float l0, l1, l2, l3;
                            unpack2(l01, l0, l1);
                            unpack2(l23, l2, l3);
                            l += (l0 + l1) + (l2 + l3);
                        }
                    } else {
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&bars->s_empty[buf]);
                    }
                }
                // the other parts of the row's columns: combine the four (maximum, sum) pairs
                tmem_st4(tmem_ml + 4 * c, m, l, 0.f, 0.f);
                tmem_wait_st();
                tmem_fence_before_sync();
                named_barrier_sync(1, kSoftmaxThreads);
                tmem_fence_after_sync();
                {
                    float pm[4], pl[4], pad0, pad1;
#pragma unroll
                    for (int k4 = 0; k4 < 4; ++k4) tmem_ld4(tmem_ml + 4 * k4, pm[k4], pl[k4], pad0, pad1);
                    tmem_wait_ld();
                    m = fmaxf(fmaxf(pm[0], pm[1]), fmaxf(pm[2], pm[3]));      // part 0 always has key 0: finite
                    l = 0.f;
#pragma unroll
                    for (int k4 = 0; k4 < 4; ++k4) l += pm[k4] > -INFINITY ? pl[k4] * fast_exp2(pm[k4] - m) : 0.f;
                }
                // rows of padded head slots get lse = +inf: all their probabilities are exactly 0
                const float lse = head_on ? m + log2f(l) : INFINITY;
                // ---- pass B: normalised probabilities back into tensor memory, pbar, activations ----
                for (int kb = 0; kb < nkb; ++kb, ++sb.count, ++tiles) {
                    const uint32_t buf = sb.stage(2);
                    wait_on(&bars->s_full[buf], sb.parity(2));
                    tmem_fence_after_sync();
                    uint32_t* act_t = act + (tiles & 1u) * kTile;
                    // the state words of the key column this lane owns, requested before the tile's arithmetic so
                    // that they are there when the activations are applied (only this thread ever writes them)
                    const int own_key = kb * kTile + c * 32 + lane;
                    int2 own = make_int2(0, 0);
                    if ((warp & 3) == 0 && own_key < P) own = p.tsm[srow + own_key];
                    const uint32_t cols = tmem_row + kColS + buf * 128 + c * 32;
                    if (kb * kTile + c * 32 > warp_last_pos) {
                        // a chunk beyond all of this warp's positions: P = 0, nothing to add up or to test
                        const uint32_t zero[16] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
                        tmem_st16(cols, zero);
                        tmem_st16(cols + 16, zero);
                        tmem_wait_st();
                        tmem_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) {
                            mbar_arrive(&bars->p_full[buf]);
                            mbar_arrive(&bars->s_empty[buf]);
                        }
                    } else {
                        float x[32];
                        tmem_ld32(cols, x);
                        tmem_wait_ld();
                        const int key0 = kb * kTile + c * 32;
                        {
                            const uint64_t scale2 = pack2(p.scale_log2, p.scale_log2), minus_lse = pack2(-lse, -lse);
#pragma unroll
                            for (int i = 0; i < 32; i += 2) {
                                float e0, e1;
                                unpack2(fma2(pack2(x[i], x[i + 1]), scale2, minus_lse), e0, e1);
                                x[i] = fast_exp2(e0);
                                x[i + 1] = fast_exp2(e1);
                            }
                        }
                        if (key0 + 31 > pos) {      // the tile on the diagonal: keys beyond the row's position weigh nothing
#pragma unroll
                            for (int i = 0; i < 32; ++i) x[i] = key0 + i <= pos ? x[i] : 0.f;
                        }
                        // P over the logits it came from, as the tensor-memory A operand of O += P V: two bf16
                        // per column, the 32 keys of this chunk as 16 columns of hi terms then 16 of lo terms
                        // (p = hi + lo, 16 mantissa bits: with one term the weights would be off by up to 2^-9,
                        // more than the output tolerance allows where large values cancel).
                        {
                            uint32_t hi[16], lo[16];
#pragma unroll
                            for (int e = 0; e < 16; ++e) {
                                const float a0 = x[2 * e], a1 = x[2 * e + 1];
                                hi[e] = pack_bf16(a0, a1);
                                float r0, r1;
                                unpack2(sub2(pack2(a0, a1), pack2(bf16_lo_as_float(hi[e]), bf16_hi_as_float(hi[e]))), r0, r1);
                                lo[e] = pack_bf16(r0, r1);
                            }
                            tmem_st16(cols, hi);
                            tmem_st16(cols + 16, lo);
                        }
                        // P is in place and the logits are in registers: hand the buffer to the tensor core now,
                        // the head sums below need nothing from tensor memory
                        tmem_wait_st();
                        tmem_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) {
                            mbar_arrive(&bars->p_full[buf]);
                            mbar_arrive(&bars->s_empty[buf]);
                        }
                        // pbar: sum over the GP lanes of this position.  Every round halves what a lane keeps,
                        // so after log2(GP) rounds lane g holds 32 / GP columns summed over all heads.
                        int col0 = 0;               // first of the columns this lane ends up with
#pragma unroll
                        for (int w = 1, half = 16; w < GP; w <<= 1, half >>= 1) {
                            const bool upper = (lane & w) != 0;
#pragma unroll
                            for (int i = 0; i < half; i += 2) {
                                const float send0 = upper ? x[i] : x[i + half], send1 = upper ? x[i + 1] : x[i + 1 + half];
                                const float keep0 = upper ? x[i + half] : x[i], keep1 = upper ? x[i + 1 + half] : x[i + 1];
                                unpack2(add2(pack2(keep0, keep1), pack2(__shfl_xor_sync(0xffffffffu, send0, w),
                                                                        __shfl_xor_sync(0xffffffffu, send1, w))),
                                        x[i], x[i + 1]);
                            }
                            col0 += upper ? half : 0;
                        }
                        constexpr int kMine = 32 / GP;
                        if (pos < P) {
#pragma unroll
                            for (int i = 0; i < kMine; ++i) {
                                const int key = key0 + col0 + i;
                                if (key <= pos) {
                                    const float pb = x[i] * p.inv_group;
                                    if (pb >= p.alpha) atomicOr(&act_t[c * 32 + col0 + i], 1u << jj);
                                    if (pos == P - 1) p.pbar[srow + key] = pb;
                                    if (dumping) p.dump[((size_t)(u - p.dump_begin) * P + pos) * P + key] = pb;
                                }
                            }
                        }
                    }
                    // Eq. (1) for this tile's activations.  The bits of the 32 columns of part c come from the four
                    // warps of part c only, so those 128 threads synchronise among themselves (the parts stay
                    // free to drift apart), and lane l of the part's first warp owns key column kb * 128 + 32 c + l.
                    named_barrier_sync(3 + c, 128);
                    const uint32_t bits = (warp & 3) == 0 ? act_t[c * 32 + lane] : 0u;
                    if (bits != 0u) {
                        act_t[c * 32 + lane] = 0u;
                        int ts = own.x, mri = own.y;
                        uint32_t left = bits;
                        while (left != 0u) {        // positions of the tile in ascending order
                            const int b = __ffs(left) - 1;
                            left &= left - 1u;
                            const int time = qt * TQ + b - (P - 1);
                            mri = max(mri, time - ts);          // MRI = max(MRI, t - TS)
                            ts = time;                          // TS = t
                        }
                        p.tsm[srow + own_key] = make_int2(ts, mri);
                    }
                }
                write_output(qr.stage(2));
            }
        }
    }

    tmem_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        tmem_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn) return fn;
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
        return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(sym);
    return fn;
}

// bf16 tensor map with 128-byte swizzle; dims / strides innermost first, strides in bytes for dims 1..rank-1.
bool make_map(CUtensorMap* map, const void* base, int rank, const cuuint64_t* dims, const cuuint64_t* strides,
              const cuuint32_t* box) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint32_t elem[5] = {1, 1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int GP>
cudaError_t launch_gp(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const CUtensorMap& mo,
                      const PromptParams& p, int blocks, cudaStream_t stream) {
    cudaError_t e = cudaFuncSetAttribute(prompt_kernel<GP>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPromptSmem);
    if (e != cudaSuccess) return e;
    prompt_kernel<GP><<<blocks, kPromptThreads, kPromptSmem, stream>>>(mq, mk, mv, mo, p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t prompt_launch(const Geometry& geo, StateView st, const PromptArgs& a, int num_sms, cudaStream_t stream) {
    const int G = geo.group, P = a.n_tokens;
    int gp = 4;                 // head slots per position: at least 4, so that a tile's positions fit a 32-bit mask
    while (gp < G) gp *= 2;
    const int tq = kTile / gp;
    CUtensorMap mq, mk, mv, mo;
    {
        // q [P][units][G][128]: box = 64 dims x GP head slots x 1 unit x TQ positions -> rows (position, head slot);
        // head slots >= G and positions >= P are outside the tensor and read as zero.
        const cuuint64_t dims[4] = {(cuuint64_t)kHeadDim, (cuuint64_t)G, (cuuint64_t)geo.units, (cuuint64_t)P};
        const cuuint64_t strides[3] = {(cuuint64_t)kRowBytes, (cuuint64_t)G * kRowBytes, (cuuint64_t)geo.units * G * kRowBytes};
        const cuuint32_t box[4] = {64, (cuuint32_t)gp, 1, (cuuint32_t)tq};
        if (!make_map(&mq, a.q, 4, dims, strides, box)) return cudaErrorInvalidValue;
        if (!make_map(&mo, a.out, 4, dims, strides, box)) return cudaErrorInvalidValue;     // out is laid out like q
    }
    {
        // k, v [units][P][128]: box = 64 dims x 128 keys x 1 unit; keys >= P read as zero.
        const cuuint64_t dims[3] = {(cuuint64_t)kHeadDim, (cuuint64_t)P, (cuuint64_t)geo.units};
        const cuuint64_t strides[2] = {(cuuint64_t)kRowBytes, (cuuint64_t)P * kRowBytes};
        const cuuint32_t box[3] = {64, (cuuint32_t)kTile, 1};
        if (!make_map(&mk, a.k, 3, dims, strides, box)) return cudaErrorInvalidValue;
        if (!make_map(&mv, a.v, 3, dims, strides, box)) return cudaErrorInvalidValue;
    }
    PromptParams p;
    p.units = geo.units;
    p.group = G;
    p.P = P;
    p.capacity = geo.capacity;
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)kHeadDim);
    p.inv_group = 1.0f / (float)G;
    p.alpha = a.alpha;
    p.tsm = st.tsm;
    p.pbar = st.pbar;
    p.status = st.status;
    p.dump = a.dump;
    p.dump_begin = a.dump_begin;
    p.dump_count = a.dump_count;
    p.wait_limit_ns = a.wait_limit_ns;
    p.stop_after_tiles = a.stop_after_tiles;
    const int blocks = geo.units < num_sms ? geo.units : num_sms;
    return gp == 4 ? launch_gp<4>(mq, mk, mv, mo, p, blocks, stream) : launch_gp<8>(mq, mk, mv, mo, p, blocks, stream);
}

}  // namespace lzk
