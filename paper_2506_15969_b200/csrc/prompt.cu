// Causal attention over the prompt with recurrence tracking from the first prompt token.
//
// For every cache unit and every prompt row j (Appendix A, Eq. (attn), with a causal mask):
//   s_g[j][i] = q_{j,g} . k_i / sqrt(D),  i <= j;   p_g[j] = softmax_i(s_g[j]);   out_{j,g} = sum_i p_g[j][i] v_i
//   pbar[j][i] = mean_g p_g[j][i]
// and, in row order (Section 4 "Recurrence Interval Tracking", Eq. (1), Algorithm 1's loop),
//   pbar[j][i] >= alpha  =>  MRI[i] = max(MRI[i], time_j - TS[i]);  TS[i] = time_j,   time_j = j - (P - 1).
//
// This is the one dense contraction of the path, so it runs on the fifth-generation tensor cores:
// tcgen05.mma with both operands in shared memory (TMA tiles, 128-byte swizzle) and accumulators in
// tensor memory.  One block owns a unit and walks its query tiles in row order; a query tile is 128
// rows = (128 / GP) prompt positions x GP query-head slots (GP = 4 or 8, the group size rounded up),
// so the heads that share the K / V tile sit in neighbouring lanes.  Every query tile makes
// two passes over its key tiles (128 keys each):
//   pass A: S = Q K^T, row maximum and sum of exponentials  ->  exact log-sum-exp per row;
//   pass B: S = Q K^T again, p = exp2(s - lse) (already normalised), P to shared memory as two bf16
//           terms (hi + lo), O += P V (no rescaling ever), pbar by a butterfly sum over the GP lanes of a position,
//           threshold test, activation bits per key column; after the tile one thread per key
//           column applies Eq. (1) for the tile's positions in ascending order.
// Key columns are owned by a fixed thread for the whole unit and query tiles are visited in ascending
// order, so every token sees its activations in row order.
//
// Warp roles: warps 0-7 softmax / tracking / epilogue (thread = accumulator row = TMEM lane; the two
// warps that share a lane quarter take one half of a tile's columns each), warp 8 TMA producer,
// warp 9 MMA issuer.  All mbarrier waits are bounded.
#include <cuda.h>

#include "internal.h"

namespace lzk {

namespace {

constexpr int kTile = 128;                         // rows of a query tile, keys of a key tile
constexpr int kBoxBytes = kTile * 128;             // one TMA box: 128 rows x 64 bf16 (16 KiB)
constexpr int kOperandBytes = 2 * kBoxBytes;       // a 128 x 128 bf16 operand tile: two boxes (32 KiB)
constexpr int kKvStages = 2;
constexpr int kSoftmaxWarps = 8;                   // two per TMEM lane quarter: each takes half of a tile's columns
constexpr int kSoftmaxThreads = 32 * kSoftmaxWarps;
constexpr int kPromptThreads = kSoftmaxThreads + 64;

// shared-memory map (offsets from a 1024-byte aligned base)
constexpr int kOffQ = 0;
constexpr int kOffKV = kOffQ + kOperandBytes;                       // per stage: K tile, then V tile
constexpr int kOffP = kOffKV + kKvStages * 2 * kOperandBytes;
constexpr int kOffMisc = kOffP + 2 * kOperandBytes;                 // P as two bf16 terms: hi tile, lo tile
constexpr int kMiscBytes = 2048;
constexpr int kPromptSmem = kOffMisc + kMiscBytes;                  // 226 KiB of the 227 KiB a block may have

struct Bars {                                       // mbarriers
    uint64_t q_full, q_empty;
    uint64_t kv_full[kKvStages], kv_empty[kKvStages];
    uint64_t s_full[2], s_empty[2];
    uint64_t p_full, p_empty;
    uint64_t o_full, o_empty;
    uint64_t drain;
};

struct PromptParams {
    int units, group, P, capacity;
    float scale_log2, inv_group, alpha;
    __nv_bfloat16* out;                             // [P][units][group][128]
    int32_t* ts;
    int32_t* mri;
    float* pbar;
    int32_t* status;
    float* dump;                                    // optional: [dump_count][P][P] probabilities per prompt row
    int dump_begin, dump_count;
    unsigned long long wait_limit_ns;
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

// Barrier over `threads` threads that also ANDs a predicate: every thread learns whether all of them
// passed their waits, so that they leave the loops together.
__device__ __forceinline__ bool named_barrier_and(int id, int threads, bool pred) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %3, 0;\n\t"
        "bar.red.and.pred p, %1, %2, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"(id), "r"(threads), "r"((uint32_t)pred)
        : "memory");
    return r != 0;
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
              const __grid_constant__ CUtensorMap map_v, const PromptParams p) {
    constexpr int TQ = kTile / GP;                  // prompt positions per query tile
    extern __shared__ __align__(1024) uint8_t smem[];           // the swizzle atoms need 1024-byte alignment
    uint8_t* q_s = smem + kOffQ;
    uint8_t* p_s = smem + kOffP;
    Bars* bars = reinterpret_cast<Bars*>(smem + kOffMisc);
    uint32_t* act = reinterpret_cast<uint32_t*>(smem + kOffMisc + 256);          // [2][128] activation bits per key column
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kOffMisc + 256 + 1024);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int P = p.P, G = p.group;

    if (threadIdx.x == 0) {
        mbar_init(&bars->q_full, 1);
        mbar_init(&bars->q_empty, 1);
        for (int i = 0; i < kKvStages; ++i) {
            mbar_init(&bars->kv_full[i], 1);
            mbar_init(&bars->kv_empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&bars->s_full[i], 1);
            mbar_init(&bars->s_empty[i], kSoftmaxWarps);
        }
        mbar_init(&bars->p_full, kSoftmaxWarps);
        mbar_init(&bars->p_empty, 1);
        mbar_init(&bars->o_full, 1);
        mbar_init(&bars->o_empty, kSoftmaxWarps);
        mbar_init(&bars->drain, 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    for (int i = threadIdx.x; i < 256; i += kPromptThreads) act[i] = 0u;
    if (warp == 0) {
        tmem_alloc(tmem_slot, 512);                 // S double buffer (2 x 128 columns) + O (128 columns)
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
            Ring kv;
            uint32_t q_uses = 0;
            bool ok = true;
            for (int u = blockIdx.x; u < p.units && ok; u += gridDim.x) {
                for (int qt = 0; qt < n_qt && ok; ++qt, ++q_uses) {
                    ok = wait_bar(&bars->q_empty, (q_uses & 1u) ^ 1u, abort_flag, p.status, limit);
                    if (!ok) break;
                    mbar_arrive_expect_tx(&bars->q_full, kOperandBytes);
                    tma_load_4d(q_s, &map_q, 0, 0, u, qt * TQ, &bars->q_full);
                    tma_load_4d(q_s + kBoxBytes, &map_q, 64, 0, u, qt * TQ, &bars->q_full);
                    const int nkb = key_tiles(qt);
                    for (int pass = 0; pass < 2 && ok; ++pass) {
                        for (int kb = 0; kb < nkb; ++kb, ++kv.count) {
                            const uint32_t st = kv.stage(kKvStages);
                            ok = wait_bar(&bars->kv_empty[st], kv.parity(kKvStages) ^ 1u, abort_flag, p.status, limit);
                            if (!ok) break;
                            uint8_t* k_s = smem + kOffKV + st * 2 * kOperandBytes;
                            mbar_arrive_expect_tx(&bars->kv_full[st], pass == 0 ? kOperandBytes : 2 * kOperandBytes);
                            tma_load_3d(k_s, &map_k, 0, kb * kTile, u, &bars->kv_full[st]);
                            tma_load_3d(k_s + kBoxBytes, &map_k, 64, kb * kTile, u, &bars->kv_full[st]);
                            if (pass == 1) {
                                tma_load_3d(k_s + kOperandBytes, &map_v, 0, kb * kTile, u, &bars->kv_full[st]);
                                tma_load_3d(k_s + kOperandBytes + kBoxBytes, &map_v, 64, kb * kTile, u, &bars->kv_full[st]);
                            }
                        }
                    }
                }
            }
            if (!ok) {
                // Aborted: let the copies already issued land before the block exits.  The loads of the
                // last kKvStages stage uses and of the last query tile may still be in flight.
                const uint32_t last = kv.count < (uint32_t)kKvStages ? kv.count : (uint32_t)kKvStages;
                for (uint32_t k = kv.count - last; k < kv.count; ++k)
                    wait_bar(&bars->kv_full[k % kKvStages], (k / kKvStages) & 1u, abort_flag, p.status, limit, false);
                if (q_uses > 0) wait_bar(&bars->q_full, (q_uses - 1) & 1u, abort_flag, p.status, limit, false);
            }
        }
    } else if (warp == kSoftmaxWarps + 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            Ring kv, sb;                            // K/V stage uses, S buffer uses
            uint32_t q_uses = 0, p_uses = 0, o_uses = 0;
            bool ok = true;
            const uint32_t idesc_s = instr_desc(false), idesc_o = instr_desc(true);
            const uint32_t q_addr = smem_u32(q_s), p_addr = smem_u32(p_s);
            const uint32_t tmem_o = tmem_base + 256;
            // S[buffer] = Q K^T for the K tile in stage `st`
            auto issue_s = [&](uint32_t st, uint32_t buf) {
                const uint32_t k_addr = smem_u32(smem + kOffKV + st * 2 * kOperandBytes);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {    // 16 head dimensions per instruction: 32 bytes inside a box row
                    const uint32_t off = (ks >> 2) * kBoxBytes + (ks & 3) * 32;
                    umma_bf16(tmem_base + buf * 128, smem_desc(q_addr + off, 16, 1024), smem_desc(k_addr + off, 16, 1024),
                              idesc_s, ks > 0);
                }
            };
            for (int u = blockIdx.x; u < p.units && ok; u += gridDim.x) {
                for (int qt = 0; qt < n_qt && ok; ++qt, ++q_uses) {
                    const int nkb = key_tiles(qt);
                    ok = wait_bar(&bars->q_full, q_uses & 1u, abort_flag, p.status, limit);
                    // pass A: logits only
                    for (int kb = 0; kb < nkb && ok; ++kb, ++kv.count, ++sb.count) {
                        const uint32_t st = kv.stage(kKvStages), buf = sb.stage(2);
                        ok = wait_bar(&bars->kv_full[st], kv.parity(kKvStages), abort_flag, p.status, limit) &&
                             wait_bar(&bars->s_empty[buf], sb.parity(2) ^ 1u, abort_flag, p.status, limit);
                        if (!ok) break;
                        tmem_fence_after_sync();
                        issue_s(st, buf);
                        umma_commit(&bars->s_full[buf]);
                        umma_commit(&bars->kv_empty[st]);
                    }
                    if (!ok) break;
                    // pass B: logits, then O += P V one key tile behind
                    ok = wait_bar(&bars->o_empty, (o_uses & 1u) ^ 1u, abort_flag, p.status, limit);
                    uint32_t st_of[2] = {0, 0};     // stage of the key tile whose P V product is still to be issued
                    for (int kb = 0; kb <= nkb && ok; ++kb) {
                        if (kb < nkb) {
                            const uint32_t st = kv.stage(kKvStages), buf = sb.stage(2);
                            ok = wait_bar(&bars->kv_full[st], kv.parity(kKvStages), abort_flag, p.status, limit) &&
                                 wait_bar(&bars->s_empty[buf], sb.parity(2) ^ 1u, abort_flag, p.status, limit);
                            if (!ok) break;
                            tmem_fence_after_sync();
                            issue_s(st, buf);
                            umma_commit(&bars->s_full[buf]);
                            st_of[kb & 1] = st;
                            ++kv.count;
                            ++sb.count;
                        }
                        if (kb > 0) {               // P of key tile kb - 1 is in shared memory
                            ok = wait_bar(&bars->p_full, p_uses & 1u, abort_flag, p.status, limit);
                            if (!ok) break;
                            tmem_fence_after_sync();
                            const uint32_t st = st_of[(kb - 1) & 1];
                            const uint32_t v_addr = smem_u32(smem + kOffKV + st * 2 * kOperandBytes + kOperandBytes);
#pragma unroll
                            for (int ks = 0; ks < 8; ++ks) {      // 16 keys per instruction; P = hi + lo, two products
                                const uint32_t a_off = (ks >> 2) * kBoxBytes + (ks & 3) * 32;
                                const uint64_t v_desc = smem_desc(v_addr + ks * 2048, kBoxBytes, 1024);
                                umma_bf16(tmem_o, smem_desc(p_addr + a_off, 16, 1024), v_desc, idesc_o, (kb > 1 || ks > 0));
                                umma_bf16(tmem_o, smem_desc(p_addr + kOperandBytes + a_off, 16, 1024), v_desc, idesc_o, 1u);
                            }
                            umma_commit(&bars->p_empty);
                            umma_commit(&bars->kv_empty[st]);
                            ++p_uses;
                        }
                    }
                    if (!ok) break;
                    umma_commit(&bars->o_full);
                    umma_commit(&bars->q_empty);
                    ++o_uses;
                }
            }
            // every MMA issued by this thread is complete before tensor memory goes back
            umma_commit(&bars->drain);
            wait_bar(&bars->drain, 0, abort_flag, p.status, limit, false);
        }
    } else {
        // ------------------------------------------------------------------ softmax, tracking, epilogue
        // Warps w and w + 4 share TMEM lanes 32 (w % 4) ..: thread = accumulator row, and the two warps of a
        // row take the lower and the upper 64 columns of every tile.
        const int row = threadIdx.x & 127;          // accumulator row = TMEM lane
        const int chalf = threadIdx.x >> 7;         // which half of the columns
        const int jj = row / GP, g = row % GP;
        const bool head_on = g < G;
        const uint32_t tmem_row = tmem_base + ((uint32_t)(32 * (warp & 3)) << 16);
        const uint32_t tmem_ml = tmem_row + 384;    // spare columns: the two halves of a row exchange (maximum, sum) here
        Ring sb;
        uint32_t p_uses = 0, o_uses = 0, tiles = 0;
        bool ok = true;
        for (int u = blockIdx.x; u < p.units && ok; u += gridDim.x) {
            const size_t srow = (size_t)u * p.capacity;
            const bool dumping = p.dump != nullptr && u >= p.dump_begin && u < p.dump_begin + p.dump_count;
            for (int qt = 0; qt < n_qt && ok; ++qt) {
                const int pos = qt * TQ + jj;
                const bool row_on = head_on && pos < P;
                const int nkb = key_tiles(qt);
                // ---- pass A: exact log-sum-exp of the row (log2 domain) ----
                float m = -INFINITY, l = 0.f;
                for (int kb = 0; kb < nkb && ok; ++kb, ++sb.count) {
                    const uint32_t buf = sb.stage(2);
                    ok = named_barrier_and(2, kSoftmaxThreads,
                                           wait_bar(&bars->s_full[buf], sb.parity(2), abort_flag, p.status, limit));
                    if (!ok) break;
                    tmem_fence_after_sync();
#pragma unroll 1
                    for (int c = 2 * chalf; c < 2 * chalf + 2; ++c) {
                        float x[32];
                        tmem_ld32(tmem_row + buf * 128 + c * 32, x);
                        tmem_wait_ld();
                        const int key0 = kb * kTile + c * 32;
                        float cmax = -INFINITY;
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            x[i] = key0 + i <= pos ? x[i] * p.scale_log2 : -INFINITY;
                            cmax = fmaxf(cmax, x[i]);
                        }
                        if (cmax > m) {
                            l *= fast_exp2(m - cmax);     // m = -inf only while l = 0
                            m = cmax;
                        }
                        if (m > -INFINITY) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) l += fast_exp2(x[i] - m);
                        }
                    }
                    tmem_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->s_empty[buf]);
                }
                if (!ok) break;
                // the row's other half of the columns: combine the two (maximum, sum) pairs
                tmem_st4(tmem_ml + 4 * chalf, m, l, 0.f, 0.f);
                tmem_wait_st();
                tmem_fence_before_sync();
                named_barrier_sync(1, kSoftmaxThreads);
                tmem_fence_after_sync();
                {
                    float om, ol, pad0, pad1;
                    tmem_ld4(tmem_ml + 4 * (chalf ^ 1), om, ol, pad0, pad1);
                    tmem_wait_ld();
                    const float mm = fmaxf(m, om);
                    l = (m > -INFINITY ? l * fast_exp2(m - mm) : 0.f) + (om > -INFINITY ? ol * fast_exp2(om - mm) : 0.f);
                    m = mm;
                }
                const float lse = m + log2f(l);
                // ---- pass B: normalised probabilities, P for the tensor core, pbar, activations ----
                for (int kb = 0; kb < nkb && ok; ++kb, ++sb.count, ++tiles) {
                    const uint32_t buf = sb.stage(2);
                    ok = named_barrier_and(2, kSoftmaxThreads,
                                           wait_bar(&bars->s_full[buf], sb.parity(2), abort_flag, p.status, limit) &&
                                               wait_bar(&bars->p_empty, (p_uses & 1u) ^ 1u, abort_flag, p.status, limit));
                    if (!ok) break;
                    tmem_fence_after_sync();
                    uint32_t* act_t = act + (tiles & 1u) * kTile;
#pragma unroll 1
                    for (int c = 2 * chalf; c < 2 * chalf + 2; ++c) {
                        float x[32];
                        tmem_ld32(tmem_row + buf * 128 + c * 32, x);
                        tmem_wait_ld();
                        const int key0 = kb * kTile + c * 32;
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            x[i] = key0 + i <= pos ? fast_exp2(x[i] * p.scale_log2 - lse) : 0.f;
                        // P as the K-major A operand of O += P V: row `row`, keys key0 .. key0 + 31 of this tile.
                        // It enters the tensor core as two bf16 terms, p = hi + lo (16 mantissa bits): with one
                        // term the weights would be off by up to 2^-9, more than the output tolerance allows
                        // where large values cancel.
                        {
                            uint8_t* prow = p_s + (c >> 1) * kBoxBytes + row * 128;
#pragma unroll
                            for (int ch = 0; ch < 4; ++ch) {
                                uint32_t hi[4], lo[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const float a0 = x[8 * ch + 2 * e], a1 = x[8 * ch + 2 * e + 1];
                                    hi[e] = pack_bf16(a0, a1);
                                    lo[e] = pack_bf16(a0 - bf16_lo_as_float(hi[e]), a1 - bf16_hi_as_float(hi[e]));
                                }
                                const int chunk = (c & 1) * 4 + ch;
                                uint8_t* dst = prow + ((chunk ^ (row & 7)) << 4);
                                *reinterpret_cast<uint4*>(dst) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                                *reinterpret_cast<uint4*>(dst + kOperandBytes) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                            }
                        }
                        // pbar: sum over the GP lanes of this position.  Every round halves what a lane keeps,
                        // so after log2(GP) rounds lane g holds 32 / GP columns summed over all heads.
                        if (!head_on) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) x[i] = 0.f;
                        }
                        int col0 = 0;               // first of the columns this lane ends up with
#pragma unroll
                        for (int w = 1, half = 16; w < GP; w <<= 1, half >>= 1) {
                            const bool upper = (lane & w) != 0;
#pragma unroll
                            for (int i = 0; i < half; ++i) {
                                const float send = upper ? x[i] : x[i + half];
                                const float keep = upper ? x[i + half] : x[i];
                                x[i] = keep + __shfl_xor_sync(0xffffffffu, send, w);
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
                    fence_proxy_async();            // P is read by the tensor core through the async proxy
                    tmem_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) {
                        mbar_arrive(&bars->p_full);
                        mbar_arrive(&bars->s_empty[buf]);
                    }
                    ++p_uses;
                    // Eq. (1) for this tile's activations: thread `row` owns key column kb * 128 + row.
                    named_barrier_sync(1, kSoftmaxThreads);
                    const uint32_t bits = chalf == 0 ? act_t[row] : 0u;
                    if (bits != 0u) {
                        act_t[row] = 0u;
                        const size_t s = srow + (size_t)kb * kTile + row;
                        int ts = p.ts[s], mri = p.mri[s];
                        uint32_t left = bits;
                        while (left != 0u) {        // positions of the tile in ascending order
                            const int b = __ffs(left) - 1;
                            left &= left - 1u;
                            const int time = qt * TQ + b - (P - 1);
                            mri = max(mri, time - ts);          // MRI = max(MRI, t - TS)
                            ts = time;                          // TS = t
                        }
                        p.ts[s] = ts;
                        p.mri[s] = mri;
                    }
                }
                if (!ok) break;
                // ---- the tile's attention output ----
                ok = named_barrier_and(2, kSoftmaxThreads, wait_bar(&bars->o_full, o_uses & 1u, abort_flag, p.status, limit));
                if (!ok) break;
                tmem_fence_after_sync();
#pragma unroll 1
                for (int c = 2 * chalf; c < 2 * chalf + 2; ++c) {
                    float x[32];
                    tmem_ld32(tmem_row + 256 + c * 32, x);
                    tmem_wait_ld();
                    if (row_on) {
                        __nv_bfloat16* orow = p.out + (((size_t)pos * p.units + u) * G + g) * kHeadDim + c * 32;
#pragma unroll
                        for (int ch = 0; ch < 4; ++ch) {
                            uint4 w;
                            w.x = pack_bf16(x[8 * ch + 0], x[8 * ch + 1]);
                            w.y = pack_bf16(x[8 * ch + 2], x[8 * ch + 3]);
                            w.z = pack_bf16(x[8 * ch + 4], x[8 * ch + 5]);
                            w.w = pack_bf16(x[8 * ch + 6], x[8 * ch + 7]);
                            *reinterpret_cast<uint4*>(orow + 8 * ch) = w;
                        }
                    }
                }
                tmem_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars->o_empty);
                ++o_uses;
            }
        }
    }

    tmem_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        tmem_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
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
cudaError_t launch_gp(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const PromptParams& p,
                      int blocks, cudaStream_t stream) {
    cudaError_t e = cudaFuncSetAttribute(prompt_kernel<GP>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPromptSmem);
    if (e != cudaSuccess) return e;
    prompt_kernel<GP><<<blocks, kPromptThreads, kPromptSmem, stream>>>(mq, mk, mv, p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t prompt_launch(const Geometry& geo, StateView st, const PromptArgs& a, int num_sms, cudaStream_t stream) {
    const int G = geo.group, P = a.n_tokens;
    int gp = 4;                 // head slots per position: at least 4, so that a tile's positions fit a 32-bit mask
    while (gp < G) gp *= 2;
    const int tq = kTile / gp;
    CUtensorMap mq, mk, mv;
    {
        // q [P][units][G][128]: box = 64 dims x GP head slots x 1 unit x TQ positions -> rows (position, head slot);
        // head slots >= G and positions >= P are outside the tensor and read as zero.
        const cuuint64_t dims[4] = {(cuuint64_t)kHeadDim, (cuuint64_t)G, (cuuint64_t)geo.units, (cuuint64_t)P};
        const cuuint64_t strides[3] = {(cuuint64_t)kRowBytes, (cuuint64_t)G * kRowBytes, (cuuint64_t)geo.units * G * kRowBytes};
        const cuuint32_t box[4] = {64, (cuuint32_t)gp, 1, (cuuint32_t)tq};
        if (!make_map(&mq, a.q, 4, dims, strides, box)) return cudaErrorInvalidValue;
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
    p.out = reinterpret_cast<__nv_bfloat16*>(a.out);
    p.ts = st.ts;
    p.mri = st.mri;
    p.pbar = st.pbar;
    p.status = st.status;
    p.dump = a.dump;
    p.dump_begin = a.dump_begin;
    p.dump_count = a.dump_count;
    p.wait_limit_ns = a.wait_limit_ns;
    const int blocks = geo.units < num_sms ? geo.units : num_sms;
    return gp == 4 ? launch_gp<4>(mq, mk, mv, p, blocks, stream) : launch_gp<8>(mq, mk, mv, p, blocks, stream);
}

}  // namespace lzk
