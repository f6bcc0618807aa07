// Host-side interfaces between the C-ABI layer and the kernel launchers.
#pragma once

#include "common.cuh"

namespace lzk {

// ---- decode ------------------------------------------------------------------
struct DecodeConfig {
    int units, group, pages_per_unit, capacity;
    float alpha;
    int force_splits;      // 0 = automatic
    int force_stages;      // 0 = automatic
    int force_groups;      // 0 = automatic; groups of four consumer warps per block (1 or 2)
    unsigned long long wait_limit_ns;   // bounded waits give up after this long
    int stop_after_pages;  // diagnostics: -1 = off
};

struct DecodePlan {
    int splits, stages, groups, pages_per_cta, logit_stride, tmem_pages, tmem_cols;
    int off_logits, off_xchg, off_wml, off_slots, off_misc, off_bars, smem_bytes;
};

struct DecodeArgs {
    const uint8_t* pool;
    StateView state;
    const void* q;
    void* out;
    int n;                 // cached tokens per unit, the new one included
    int t;                 // this decode step
    int unit_begin, unit_count;   // the units this launch covers
    int rounds_before;            // whole rounds of the same walk done by earlier launches (0 for a walk of its own)
    const void* k_new;            // non-null: the launch also appends the new token (slot n - 1, TS = t, MRI = 0)
    const void* v_new;
    int append_position;
};

// Deepest ring and the shared-memory layout for n cached tokens and a cluster of `splits` blocks;
// -1 if nothing fits.
int decode_plan(const DecodeConfig& c, int n, int max_smem, int splits, DecodePlan* plan);
cudaError_t decode_prepare();
cudaError_t decode_max_clusters(const DecodePlan& plan, int* clusters);
cudaError_t decode_launch(const DecodeConfig& c, const DecodePlan& plan, int clusters, const DecodeArgs& a,
                          cudaStream_t stream);

// ---- cache maintenance ---------------------------------------------------------
cudaError_t init_state_launch(const Geometry& geo, StateView st, cudaStream_t stream);
// ts_first = INT_MIN: every prompt token starts at TS = 0; otherwise token i starts at TS = ts_first + i.
cudaError_t prefill_launch(const Geometry& geo, uint8_t* pool, StateView st, const void* k, const void* v,
                           int n_tokens, int ts_first, cudaStream_t stream);
cudaError_t append_launch(const Geometry& geo, uint8_t* pool, StateView st, const void* k_new, const void* v_new,
                          int slot, int t, int position, cudaStream_t stream);

// ---- prompt pass (causal attention over the prompt with tracking) -----------------------------------
struct PromptArgs {
    const void* q;         // [P][units][group][128] bf16
    const void* k;         // [units][P][128] bf16
    const void* v;
    void* out;             // like q
    int n_tokens;          // P
    float alpha;
    float* dump;           // optional [dump_count][P][P] probabilities per prompt row
    int dump_begin, dump_count;
    unsigned long long wait_limit_ns;
    int stop_after_tiles;  // diagnostics: starve the K-tile ring (-1: off)
};
// TS / MRI of the prompt tokens must already hold their starting values (TS = own time, MRI = 0).
cudaError_t prompt_launch(const Geometry& geo, StateView st, const PromptArgs& a, int num_sms, cudaStream_t stream);

// ---- eviction --------------------------------------------------------------------
struct EvictArgs {
    int n;                 // cached tokens before the eviction
    int budget;            // tokens to keep (B_t)
    int n_recent, n_initial;
    int t;
    int score_mode;
    int32_t* src;          // [units][budget]: slot that moves to slot j
    int32_t* first_moved;  // [units]: first j with src[j] != j (budget if none)
    const double* h2_table;   // H2 term of the score per MRI value, for the mode in score_mode
    int h2_entries;
    int32_t* radix_list;   // [units]: units whose k-th score is not zero (filled by the first select stage)
    int32_t* radix_count;  // [1]
};

constexpr int kH2TableEntries = 1 << 15;    // MRI values covered by the table; larger ones are evaluated directly
// Fills table[m], m < entries, with the H2 term of Eq. (2) in the variant `score_mode` selects.
cudaError_t h2_table_launch(int score_mode, int entries, double* table, cudaStream_t stream);

size_t select_smem_bytes(int n_candidates);
cudaError_t select_prepare();
cudaError_t select_launch(const Geometry& geo, StateView st, const EvictArgs& a, int num_sms, cudaStream_t stream);
cudaError_t compact_launch(const Geometry& geo, uint8_t* pool, StateView st, const EvictArgs& a,
                           cudaStream_t stream);
// Eq. (2) for every slot < n of units [unit_begin, unit_begin + unit_count) into out[unit][capacity].
cudaError_t score_launch(const Geometry& geo, StateView st, int unit_begin, int unit_count, int n, int t,
                         int score_mode, double* out, cudaStream_t stream);

// hist[b] (b < bins - 1) = cached tokens of the unit range with MRI = b; hist[bins - 1] = the rest.
cudaError_t mri_histogram_launch(const Geometry& geo, StateView st, int unit_begin, int unit_count, int n, int bins,
                                 unsigned long long* hist, cudaStream_t stream);

}  // namespace lzk
