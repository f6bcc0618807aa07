// C-ABI layer: host-side handle, argument validation, step / eviction schedule, launches.
#include <limits.h>
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <map>
#include <utility>
#include <vector>

#include "../../include/lazyev.h"
#include "internal.h"

using namespace lzk;

constexpr int kHostChunks = 3;            // unit ranges the host-buffer entry point pipelines copies over

struct lazyev {
    // configuration
    int layers = 0, batch = 1, q_heads = 0, kv_heads = 0, head_dim = 0;
    int budget = 0, budget_now = 0, window = 0, n_recent = 0, n_initial = 0, max_prefill = 0;
    float alpha = 0.f;
    int auto_evict = 1, score_mode = LAZYEV_SCORE_H1_PLUS_H2, force_splits = 0, force_stages = 0, force_groups = 0;
    int prompt_mode = LAZYEV_PROMPT_TILED;
    float* prompt_dump = nullptr;          // optional per-row probabilities of the prompt pass (caller's device memory)
    int prompt_dump_begin = 0, prompt_dump_count = 0;
    unsigned long long wait_limit_ns = 2000000000ull;   // bounded waits in the kernels give up after this long
    int stop_after_pages = -1;             // diagnostics: starve the decode kernel's page ring (-1: off)
    int fuse_append = 1;                   // small problems: the append runs inside the decode launch
    // derived at bind
    bool bound = false, prefilled = false;
    int units = 0, group = 0, capacity = 0, pages_per_unit = 0;
    int device = -1, num_sms = 0, max_smem = 0;
    cudaStream_t stream = nullptr;
    uint8_t* pool = nullptr;
    StateView st = {};
    int32_t* src = nullptr;
    int32_t* first_moved = nullptr;
    int32_t* radix_list = nullptr;         // [units] + the counter behind it
    // staging of the host-buffer entry points: two slots, so that the copies of one step run beside
    // the kernels of the step before it
    uint8_t* stage_q[2] = {nullptr, nullptr};
    uint8_t* stage_k[2] = {nullptr, nullptr};
    uint8_t* stage_v[2] = {nullptr, nullptr};
    uint8_t* stage_out[2] = {nullptr, nullptr};
    double* stage_score = nullptr;
    unsigned long long* stage_hist = nullptr;
    double* h2_table = nullptr;            // H2 term per MRI value (scratch), valid for h2_table_mode
    int h2_table_mode = -1;
    // host-buffer entry point: copy streams and events, created at its first call
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    // second launch of a step (the partly filled last round) runs beside the end of the main launch
    cudaStream_t tail_stream = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    cudaEvent_t ev_in[kHostChunks + 1] = {}, ev_done[kHostChunks + 1] = {}, ev_ready = nullptr;
    // asynchronous host-buffer steps: completion event per staging slot, steps queued so far, and
    // whether the slot's last step may still be in flight
    cudaEvent_t ev_step_done[2] = {nullptr, nullptr};
    long long host_seq = 0;
    bool slot_busy[2] = {false, false};
    int last_host_ranges = 0;
    // progress
    int t = 0, n = 0, prefill = 0;
    long long launches = 0, evictions = 0;
    DecodePlan last_plan = {};
    int last_grid = 0, last_tail_units = 0, last_tail_splits = 0;
    struct Shape {
        int splits = 1, clusters = 1, tail_splits = 0, tail_units = 0, forced_splits = 0, forced_stages = 0, forced_groups = 0;
    };
    std::map<int, Shape> plan_cache;                       // pages in use -> launch shape
    // optional per-kernel timing with CUDA events
    struct Span {
        cudaEvent_t start, stop;
        int kind;
        double bytes;
    };
    bool profiling = false;
    std::vector<Span> pending;
    std::vector<cudaEvent_t> free_events;
    lazyev_profile_t prof = {};
    char err[256] = {0};
};

namespace {

constexpr int kScoreStageUnits = 32;      // units whose scores one dump pass evaluates
constexpr int kMaxHistBins = 1 << 16;     // bins of lazyev_mri_histogram()

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int fail(lazyev_t* h, int code, const char* fmt, ...) {
    if (h) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(h->err, sizeof(h->err), fmt, ap);
        va_end(ap);
    }
    return code;
}

int cuda_fail(lazyev_t* h, cudaError_t e, const char* what) {
    return fail(h, LAZYEV_ECUDA, "%s: %s", what, cudaGetErrorString(e));
}

void derive(lazyev_t* h) {
    h->units = h->layers * h->batch * h->kv_heads;
    h->group = h->q_heads / h->kv_heads;
    const int cap = (h->budget > h->max_prefill ? h->budget : h->max_prefill) + h->window;
    h->pages_per_unit = (cap + kPageTokens - 1) / kPageTokens;
    h->capacity = h->pages_per_unit * kPageTokens;
}

struct Sizes {
    size_t kv, state, scratch;
    size_t off_tsm, off_pos, off_pbar, off_status;                                  // inside state
    size_t off_first, off_rlist, off_q, off_k, off_v, off_out, off_score, off_hist, off_h2;    // inside scratch
};

Sizes sizes_of(const lazyev_t* h) {
    Sizes s;
    const size_t slots = (size_t)h->units * h->capacity;
    s.kv = (size_t)h->units * h->pages_per_unit * kPageBytes;
    size_t off = align_up((size_t)h->units * h->pages_per_unit * sizeof(int32_t), 256);
    s.off_tsm = off;                       // (TS, MRI) pairs
    off += align_up(slots * 8, 256);
    s.off_pos = off;
    off += align_up(slots * 4, 256);
    s.off_pbar = off;
    off += align_up(slots * 4, 256);
    s.off_status = off;
    off += 256;
    s.state = off;
    off = align_up((size_t)h->units * h->budget * sizeof(int32_t), 256);
    s.off_first = off;
    off += align_up((size_t)h->units * sizeof(int32_t), 256);
    s.off_rlist = off;
    off += align_up(((size_t)h->units + 1) * sizeof(int32_t), 256);
    const size_t qbytes = (size_t)h->layers * h->batch * h->q_heads * kRowBytes;
    const size_t kbytes = (size_t)h->layers * h->batch * h->kv_heads * kRowBytes;
    s.off_q = off;                          // each staging area holds two slots
    off += 2 * align_up(qbytes, 256);
    s.off_k = off;
    off += 2 * align_up(kbytes, 256);
    s.off_v = off;
    off += 2 * align_up(kbytes, 256);
    s.off_out = off;
    off += 2 * align_up(qbytes, 256);
    s.off_score = off;
    off += align_up((size_t)kScoreStageUnits * h->capacity * sizeof(double), 256);
    s.off_hist = off;
    off += align_up((size_t)kMaxHistBins * sizeof(unsigned long long), 256);
    s.off_h2 = off;
    off += align_up((size_t)kH2TableEntries * sizeof(double), 256);
    s.scratch = off;
    return s;
}

Geometry geometry(const lazyev_t* h) { return Geometry{h->units, h->group, h->pages_per_unit, h->capacity}; }

int check_device_status(lazyev_t* h) {
    int32_t status = 0;
    cudaError_t e = cudaMemcpyAsync(&status, h->st.status, sizeof(status), cudaMemcpyDeviceToHost, h->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
    if (e != cudaSuccess) return cuda_fail(h, e, "reading the device status word");
    if (status != 0) return fail(h, LAZYEV_EDEVICE, "device status word = %d (1: wait timed out, 2: bad index)", status);
    return LAZYEV_OK;
}

enum { kSpanAppend = 0, kSpanDecode = 1, kSpanSelect = 2, kSpanCompact = 3 };

cudaEvent_t take_event(lazyev_t* h) {
    if (!h->free_events.empty()) {
        cudaEvent_t e = h->free_events.back();
        h->free_events.pop_back();
        return e;
    }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
}

// Brackets one kernel launch with events when profiling is on.
struct SpanGuard {
    lazyev_t* h;
    lazyev::Span span;
    bool on;
    SpanGuard(lazyev_t* h_, int kind, double bytes) : h(h_), on(h_->profiling) {
        if (!on) return;
        span.start = take_event(h);
        span.stop = take_event(h);
        span.kind = kind;
        span.bytes = bytes;
        cudaEventRecord(span.start, h->stream);
    }
    ~SpanGuard() {
        if (!on) return;
        cudaEventRecord(span.stop, h->stream);
        h->pending.push_back(span);
    }
};

int collect_profile(lazyev_t* h) {
    if (h->pending.empty()) return LAZYEV_OK;
    cudaError_t e = cudaStreamSynchronize(h->stream);
    if (e != cudaSuccess) return cuda_fail(h, e, "stream synchronisation");
    for (const lazyev::Span& sp : h->pending) {
        float ms = 0.f;
        cudaEventElapsedTime(&ms, sp.start, sp.stop);
        switch (sp.kind) {
            case kSpanAppend: h->prof.append_ms += ms; h->prof.append_launches++; break;
            case kSpanDecode: h->prof.decode_ms += ms; h->prof.decode_launches++; h->prof.decode_bytes += sp.bytes; break;
            case kSpanSelect: h->prof.select_ms += ms; h->prof.select_launches++; h->prof.select_bytes += sp.bytes; break;
            default: h->prof.compact_ms += ms; h->prof.compact_launches++; break;
        }
        h->free_events.push_back(sp.start);
        h->free_events.push_back(sp.stop);
    }
    h->pending.clear();
    return LAZYEV_OK;
}

// Candidates of an eviction over n cached tokens, or -1 when the select kernel cannot hold them.
int candidates_of(const lazyev_t* h, int n) {
    const int ncand = n - h->n_recent - h->n_initial;
    if (ncand <= 0 || select_smem_bytes(ncand) > 200 * 1024) return -1;
    return ncand;
}

bool evict_due_at(const lazyev_t* h, int t, int n) { return t != 0 && t % h->window == 0 && n > h->budget_now; }

// The lagged eviction of Section 4 at the current step, if one is due.  `src` and `first_moved` are
// the work lists of the select and compact kernels: the bound scratch region's or the library's own.
int run_evict(lazyev_t* h, int* evicted, int32_t* src, int32_t* first_moved, int32_t* radix_list) {
    if (evicted) *evicted = 0;
    if (!evict_due_at(h, h->t, h->n)) return LAZYEV_OK;
    const int ncand = candidates_of(h, h->n);
    if (ncand < 0)
        return fail(h, LAZYEV_EINVAL, "eviction over %d candidates is not supported", h->n - h->n_recent - h->n_initial);
    cudaError_t e;
    if (h->h2_table_mode != h->score_mode) {      // the H2 term per MRI value, in the variant the mode selects
        e = h2_table_launch(h->score_mode, kH2TableEntries, h->h2_table, h->stream);
        if (e != cudaSuccess) return cuda_fail(h, e, "H2 table launch");
        h->h2_table_mode = h->score_mode;
        h->launches += 1;
    }
    EvictArgs a;
    a.n = h->n;
    a.budget = h->budget_now;
    a.n_recent = h->n_recent;
    a.n_initial = h->n_initial;
    a.t = h->t;
    a.score_mode = h->score_mode;
    a.src = src;
    a.first_moved = first_moved;
    a.h2_table = h->h2_table;
    a.h2_entries = kH2TableEntries;
    a.radix_list = radix_list;
    a.radix_count = radix_list + h->units;
    const Geometry geo = geometry(h);
    {
        // algorithmic bytes: TS and MRI of every candidate read, the source list written
        SpanGuard g(h, kSpanSelect, (double)h->units * (8.0 * ncand + 4.0 * a.budget));
        e = select_launch(geo, h->st, a, h->num_sms, h->stream);
    }
    if (e != cudaSuccess) return cuda_fail(h, e, "select kernel launch");
    h->launches += 1;        // the selection is two launches
    {
        SpanGuard g(h, kSpanCompact, 0.0);
        e = compact_launch(geo, h->pool, h->st, a, h->stream);
    }
    if (e != cudaSuccess) return cuda_fail(h, e, "compact kernel launch");
    h->launches += 2;
    h->evictions += 1;
    if (evicted) *evicted = h->n - h->budget_now;
    h->n = h->budget_now;
    if (h->profiling) {
        // rows that actually moved: every destination from the first evicted slot on
        std::vector<int32_t> first(h->units);
        e = cudaMemcpyAsync(first.data(), first_moved, first.size() * 4, cudaMemcpyDeviceToHost, h->stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
        if (e != cudaSuccess) return cuda_fail(h, e, "first_moved download");
        double rows = 0;
        for (int32_t f : first) rows += a.budget - f;
        // per moved row: K and V rows and three state words read and written, one source index read
        h->prof.compact_bytes += rows * (2.0 * (2 * kRowBytes + 12) + 4.0);
        h->prof.compact_rows += rows;
    }
    return LAZYEV_OK;
}

// Host side of a pipelined step: queries come from and outputs go to host memory in unit ranges, on
// two copy streams, while the decode launches of the other ranges run.
struct HostPipe {
    const uint8_t* q_host;
    uint8_t* out_host;
};

// The new token of a step (S1), when the step has one.
struct NewToken {
    const void* k;
    const void* v;
    int position;
};

// The decode launches of one step: attention of q over the first n cached tokens of every unit with
// tracking at time t.  `tok` (may be null) is the token to append at slot n - 1 first: as a launch of
// its own, or -- when every block of the decode launch takes exactly one unit, the launch-latency-sized
// problems -- inside the decode launch.
int run_decode(lazyev_t* h, const void* q, void* out, int n, int t, const HostPipe* pipe, const NewToken* tok = nullptr) {
    cudaError_t e = cudaSuccess;
    DecodeConfig c{h->units, h->group, h->pages_per_unit, h->capacity, h->alpha, h->force_splits, h->force_stages, h->force_groups,
                   h->wait_limit_ns, h->stop_after_pages};
    // Launch shape, chosen per number of pages in use and cached.  For every cluster size whose logits
    // fit, a small time model gives the time of the rounds of the round-robin walk; the main launch is
    // the size with the least total.  A partly filled last round goes to a second launch with larger
    // clusters when that is faster, so that more SMs share its units.
    const int np = (n + kPageTokens - 1) / kPageTokens;
    auto cached = h->plan_cache.find(np);
    if (cached == h->plan_cache.end() || cached->second.forced_splits != h->force_splits ||
        cached->second.forced_stages != h->force_stages || cached->second.forced_groups != h->force_groups) {
        lazyev::Shape best;
        best.forced_splits = h->force_splits;
        best.forced_stages = h->force_stages;
        best.forced_groups = h->force_groups;
        // Time model, in units of the time one block needs for one page when it is not limited by HBM
        // (fitted on B200 at 8 k tokens per unit): a round of `m` units on clusters of s blocks takes
        //   max(pages per block + kFixedPages, kHbmPageTime * m * np / SMs) / ring weight
        // -- a fixed cost per unit (merge, pipeline refill), and the HBM floor once many SMs stream; a second
        // launch costs kSecondLaunchPages on top of its round.
        static const double kRingWeight[7] = {0, 0, 0.70, 0.90, 0.96, 0.99, 1.0};
        constexpr double kFixedPages = 8.0, kHbmPageTime = 1.12, kSecondLaunchPages = 10.0;
        int max_clusters[9] = {0}, stages_of[9] = {0};
        for (int s = 1; s <= 8; ++s) {
            if (h->force_splits == 0 && s > 1 && (np < 2 * s)) continue;       // at least two pages per block
            DecodePlan plan;
            if (decode_plan(c, n + kPageTokens, h->max_smem, s, &plan) != 0) continue;   // room for the page count to grow by one
            int clusters = 0;
            e = decode_max_clusters(plan, &clusters);
            if (e != cudaSuccess) {
                cudaGetLastError();
                continue;
            }
            max_clusters[s] = clusters;
            stages_of[s] = plan.stages;
        }
        auto round_time = [&](int s, int m) {
            const double own = (double)((np + s - 1) / s) + kFixedPages;
            const double hbm = kHbmPageTime * (double)m * np / h->num_sms;
            return (own > hbm ? own : hbm) / kRingWeight[stages_of[s]];
        };
        double best_time = -1.0;
        for (int s = 1; s <= 8; ++s) {
            if (max_clusters[s] < 1 || (h->force_splits > 0 && s != h->force_splits)) continue;
            const int used = max_clusters[s] < h->units ? max_clusters[s] : h->units;
            const int full = h->units / used, rem = h->units % used;
            double time = full * round_time(s, used);
            int ts = 0;
            if (rem > 0) {
                // the partly filled last round: as it is, or in a second launch with larger clusters
                double tail = round_time(s, rem);
                if (full > 0 && h->force_splits == 0)
                    for (int k = s + 1; k <= 8; ++k)
                        if (max_clusters[k] >= rem && rem * k <= h->num_sms &&
                            round_time(k, rem) + kSecondLaunchPages < tail) {
                            tail = round_time(k, rem) + kSecondLaunchPages;
                            ts = k;
                        }
                time += tail;
            }
            if (best_time < 0 || time < 0.98 * best_time) {      // larger clusters only for a clear gain
                best_time = time;
                best.splits = s;
                best.clusters = used;
                best.tail_splits = ts;
                best.tail_units = ts > 0 ? rem : 0;
            }
        }
        if (best_time < 0) return fail(h, LAZYEV_EINVAL, "no decode launch shape fits %d tokens per unit in shared memory", n);
        cached = h->plan_cache.insert_or_assign(np, best).first;
    }
    const lazyev::Shape shape = cached->second;
    DecodePlan plan;
    if (decode_plan(c, n, h->max_smem, shape.splits, &plan) != 0)
        return fail(h, LAZYEV_EINVAL, "no decode launch shape fits %d tokens per unit in shared memory", n);
    DecodePlan tail_plan = {};
    if (shape.tail_units > 0 && decode_plan(c, n, h->max_smem, shape.tail_splits, &tail_plan) != 0)
        return fail(h, LAZYEV_EINVAL, "no decode launch shape fits %d tokens per unit in shared memory", n);
    const int main_units = h->units - shape.tail_units;
    const int clusters = shape.clusters < main_units ? shape.clusters : main_units;
    const bool fuse_append = tok && h->fuse_append && shape.tail_units == 0 && main_units <= clusters;
    if (tok && !fuse_append) {
        SpanGuard g(h, kSpanAppend, 0.0);
        e = append_launch(geometry(h), h->pool, h->st, tok->k, tok->v, n - 1, t, tok->position, h->stream);
        if (e != cudaSuccess) return cuda_fail(h, e, "append kernel launch");
        h->launches += 1;
    }
    {
        // algorithmic bytes: every cached K and V row read once, one probability written per token,
        // the queries read and the outputs written
        SpanGuard g(h, kSpanDecode, (double)h->units * ((double)n * (2 * kRowBytes + 4) + 2.0 * h->group * kRowBytes));
        // Unit ranges: the main launch as one range, or (host buffers) as up to kHostChunks ranges of whole
        // rounds so that copies of one range overlap the kernel of another; then the last round's units.
        int begin[kHostChunks + 1], count[kHostChunks + 1], ranges = 0;
        const int rounds = (main_units + clusters - 1) / clusters;
        // (short first and last ranges: the first query copy and the last output copy are not overlapped)
        static const int kShare[kHostChunks + 1] = {0, 1, 11, 12};       // cumulative twelfths of the rounds
        const bool split = pipe && rounds >= 12;
        const int parts = split ? kHostChunks : 1;
        for (int r = 0; r < parts; ++r) {
            const int b = split ? rounds * kShare[r] / 12 * clusters : 0;
            int e2 = split ? rounds * kShare[r + 1] / 12 * clusters : main_units;
            if (e2 > main_units) e2 = main_units;
            if (e2 <= b) continue;
            begin[ranges] = b;
            count[ranges++] = e2 - b;
        }
        if (shape.tail_units > 0) {
            begin[ranges] = main_units;
            count[ranges++] = shape.tail_units;
        }
        const size_t unit_bytes = (size_t)h->group * kRowBytes;
        if (pipe) h->last_host_ranges = ranges;
        if (pipe) {
            for (int r = 0; r < ranges && e == cudaSuccess; ++r) {
                e = cudaMemcpyAsync((uint8_t*)const_cast<void*>(q) + begin[r] * unit_bytes, pipe->q_host + begin[r] * unit_bytes,
                                    count[r] * unit_bytes, cudaMemcpyHostToDevice, h->copy_in);
                if (e == cudaSuccess) e = cudaEventRecord(h->ev_in[r], h->copy_in);
            }
        }
        // The last round's units do not depend on the main launch: on a lower-priority stream of their own,
        // forked here (after the append), their blocks take the SMs that the main launch's blocks leave as
        // they finish; the bound stream joins afterwards.
        const bool fork = shape.tail_units > 0 && !pipe && ranges > 1;
        if (fork) {
            if (!h->tail_stream) {
                int lo = 0, hi = 0;
                e = cudaDeviceGetStreamPriorityRange(&lo, &hi);
                if (e == cudaSuccess) e = cudaStreamCreateWithPriority(&h->tail_stream, cudaStreamNonBlocking, lo);
                if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming);
                if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming);
            }
            if (e == cudaSuccess) e = cudaEventRecord(h->ev_fork, h->stream);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(h->tail_stream, h->ev_fork, 0);
        }
        for (int r = 0; r < ranges && e == cudaSuccess; ++r) {
            const bool is_tail = shape.tail_units > 0 && r == ranges - 1;
            if (pipe) e = cudaStreamWaitEvent(h->stream, h->ev_in[r], 0);
            if (e != cudaSuccess) break;
            // a range of the main walk continues it; the last round's units are a walk of their own
            DecodeArgs a{h->pool, h->st, q, out, n, t, begin[r], count[r], is_tail ? 0 : begin[r] / clusters,
                         fuse_append ? tok->k : nullptr, fuse_append ? tok->v : nullptr, fuse_append ? tok->position : 0};
            const bool beside = is_tail && fork;
            if (e != cudaSuccess) break;
            e = decode_launch(c, is_tail ? tail_plan : plan, is_tail ? count[r] : (clusters < count[r] ? clusters : count[r]), a,
                              beside ? h->tail_stream : h->stream);
            h->launches += 1;
            if (beside && e == cudaSuccess) {
                e = cudaEventRecord(h->ev_join, h->tail_stream);
                if (e == cudaSuccess) e = cudaStreamWaitEvent(h->stream, h->ev_join, 0);
            }
            if (pipe && e == cudaSuccess) {
                e = cudaEventRecord(h->ev_done[r], h->stream);
                if (e == cudaSuccess) e = cudaStreamWaitEvent(h->copy_out, h->ev_done[r], 0);
                if (e == cudaSuccess)
                    e = cudaMemcpyAsync(pipe->out_host + begin[r] * unit_bytes, (uint8_t*)out + begin[r] * unit_bytes,
                                        count[r] * unit_bytes, cudaMemcpyDeviceToHost, h->copy_out);
            }
        }
    }
    if (e != cudaSuccess) return cuda_fail(h, e, "decode kernel launch");
    h->last_plan = plan;
    h->last_tail_units = shape.tail_units;
    h->last_tail_splits = shape.tail_splits;
    h->last_grid = clusters * plan.splits;
    return LAZYEV_OK;
}

int run_step(lazyev_t* h, const void* q, const void* k_new, const void* v_new, void* out, const HostPipe* pipe = nullptr) {
    if (!h->prefilled) return fail(h, LAZYEV_ESTATE, "decode_step before prefill");
    if (h->n + 1 > h->capacity) return fail(h, LAZYEV_ECAPACITY, "cache full (%d slots per unit)", h->capacity);
    const int t = h->t + 1, n = h->n + 1;
    // A step whose automatic eviction could not run is refused before anything is queued.
    if (h->auto_evict && evict_due_at(h, t, n) && candidates_of(h, n) < 0)
        return fail(h, LAZYEV_EINVAL,
                    "step %d would evict over %d candidates, more than the selection supports; nothing was done", t,
                    n - h->n_recent - h->n_initial);
    const NewToken tok{k_new, v_new, h->prefill + t - 1};
    const int rc = run_decode(h, q, out, n, t, pipe, &tok);
    if (rc != LAZYEV_OK) return rc;
    h->t = t;
    h->n = n;
    if (h->auto_evict) return run_evict(h, nullptr, h->src, h->first_moved, h->radix_list);
    return LAZYEV_OK;
}

}  // namespace

extern "C" {

const char* lazyev_strerror(int code) {
    switch (code) {
        case LAZYEV_OK: return "ok";
        case LAZYEV_EINVAL: return "invalid argument";
        case LAZYEV_ESTATE: return "call made in the wrong state";
        case LAZYEV_ECAPACITY: return "cache capacity exceeded";
        case LAZYEV_EDEVICE: return "device-side failure flagged";
        case LAZYEV_ECUDA: return "CUDA runtime error";
        default: return "unknown error code";
    }
}

const char* lazyev_last_error(const lazyev_t* h) { return h ? h->err : "null handle"; }

int lazyev_build_flags(void) { return kBuildFlags; }

int lazyev_create(lazyev_t** handle, int layers, int q_heads, int kv_heads, int head_dim, int budget, int window,
                  float threshold) {
    if (!handle) return LAZYEV_EINVAL;
    *handle = nullptr;
    if (layers <= 0 || q_heads <= 0 || kv_heads <= 0 || budget <= 0 || window <= 0) return LAZYEV_EINVAL;
    if (head_dim != kHeadDim) return LAZYEV_EINVAL;
    if (q_heads % kv_heads != 0 || q_heads / kv_heads > kMaxGroup) return LAZYEV_EINVAL;
    if (budget <= window) return LAZYEV_EINVAL;
    if (!(threshold >= 0.f)) return LAZYEV_EINVAL;
    lazyev_t* h = new (std::nothrow) lazyev();
    if (!h) return LAZYEV_EINVAL;
    h->layers = layers;
    h->q_heads = q_heads;
    h->kv_heads = kv_heads;
    h->head_dim = head_dim;
    h->budget = h->budget_now = h->max_prefill = budget;
    h->window = window;
    h->n_recent = window;
    h->alpha = threshold;
    derive(h);
    *handle = h;
    return LAZYEV_OK;
}

int lazyev_set_batch(lazyev_t* h, int batch) {
    if (!h) return LAZYEV_EINVAL;
    if (h->bound) return fail(h, LAZYEV_ESTATE, "set_batch after bind");
    if (batch <= 0) return fail(h, LAZYEV_EINVAL, "batch must be positive");
    h->batch = batch;
    derive(h);
    return LAZYEV_OK;
}

int lazyev_set_protect(lazyev_t* h, int n_recent, int n_initial) {
    if (!h) return LAZYEV_EINVAL;
    if (h->bound) return fail(h, LAZYEV_ESTATE, "set_protect after bind");
    if (n_recent < 1 || n_initial < 0 || h->budget <= n_recent + n_initial)
        return fail(h, LAZYEV_EINVAL, "need n_recent >= 1, n_initial >= 0 and budget > n_recent + n_initial");
    h->n_recent = n_recent;
    h->n_initial = n_initial;
    return LAZYEV_OK;
}

int lazyev_set_max_prefill(lazyev_t* h, int n_tokens) {
    if (!h) return LAZYEV_EINVAL;
    if (h->bound) return fail(h, LAZYEV_ESTATE, "set_max_prefill after bind");
    if (n_tokens <= 0) return fail(h, LAZYEV_EINVAL, "max_prefill must be positive");
    h->max_prefill = n_tokens;
    derive(h);
    return LAZYEV_OK;
}

int lazyev_set_budget(lazyev_t* h, int budget_now) {
    if (!h) return LAZYEV_EINVAL;
    if (budget_now <= h->n_recent + h->n_initial || budget_now > h->budget)
        return fail(h, LAZYEV_EINVAL, "budget_now must be in (n_recent + n_initial, budget]");
    h->budget_now = budget_now;
    return LAZYEV_OK;
}

int lazyev_set_auto_evict(lazyev_t* h, int on) {
    if (!h) return LAZYEV_EINVAL;
    h->auto_evict = on != 0;
    return LAZYEV_OK;
}

int lazyev_set_score_mode(lazyev_t* h, int mode) {
    if (!h) return LAZYEV_EINVAL;
    if (mode < 0 || mode > 3) return fail(h, LAZYEV_EINVAL, "unknown score mode %d", mode);
    h->score_mode = mode;
    return LAZYEV_OK;
}

int lazyev_set_splits(lazyev_t* h, int splits) {
    if (!h) return LAZYEV_EINVAL;
    if (splits < 0 || splits > 8) return fail(h, LAZYEV_EINVAL, "splits must be 0 (automatic) or 1..8");
    h->force_splits = splits;
    return LAZYEV_OK;
}

int lazyev_set_stages(lazyev_t* h, int stages) {
    if (!h) return LAZYEV_EINVAL;
    if (stages != 0 && (stages < 2 || stages > 6)) return fail(h, LAZYEV_EINVAL, "stages must be 0 or 2..6");
    h->force_stages = stages;
    return LAZYEV_OK;
}

int lazyev_set_groups(lazyev_t* h, int groups) {
    if (!h) return LAZYEV_EINVAL;
    if (groups < 0 || groups > 2) return fail(h, LAZYEV_EINVAL, "groups must be 0 (automatic), 1 or 2");
    h->force_groups = groups;
    return LAZYEV_OK;
}

int lazyev_query_sizes(const lazyev_t* h, size_t* kv_bytes, size_t* state_bytes, size_t* scratch_bytes) {
    if (!h) return LAZYEV_EINVAL;
    const Sizes s = sizes_of(h);
    if (kv_bytes) *kv_bytes = s.kv;
    if (state_bytes) *state_bytes = s.state;
    if (scratch_bytes) *scratch_bytes = s.scratch;
    return LAZYEV_OK;
}

int lazyev_bind(lazyev_t* h, void* kv_pool, void* state, void* scratch, void* cuda_stream) {
    if (!h) return LAZYEV_EINVAL;
    if (h->bound) return fail(h, LAZYEV_ESTATE, "already bound");
    if (!kv_pool || !state || !scratch) return fail(h, LAZYEV_EINVAL, "null device pointer");
    if (((uintptr_t)kv_pool | (uintptr_t)state | (uintptr_t)scratch) & 255)
        return fail(h, LAZYEV_EINVAL, "device regions must be 256-byte aligned");
    cudaError_t e = cudaGetDevice(&h->device);
    if (e != cudaSuccess) return cuda_fail(h, e, "cudaGetDevice");
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, h->device);
    if (e != cudaSuccess) return cuda_fail(h, e, "cudaGetDeviceProperties");
    if (prop.major != 10) return fail(h, LAZYEV_ECUDA, "this library is built for sm_100a only (device is sm_%d%d)", prop.major, prop.minor);
    h->num_sms = prop.multiProcessorCount;
    h->max_smem = (int)prop.sharedMemPerBlockOptin;
    if ((e = decode_prepare()) != cudaSuccess) return cuda_fail(h, e, "decode kernel set-up");
    if ((e = select_prepare()) != cudaSuccess) return cuda_fail(h, e, "select kernel set-up");

    const Sizes s = sizes_of(h);
    h->stream = (cudaStream_t)cuda_stream;
    h->pool = (uint8_t*)kv_pool;
    uint8_t* sp = (uint8_t*)state;
    h->st.page_table = (int32_t*)sp;
    h->st.tsm = (int2*)(sp + s.off_tsm);
    h->st.pos = (int32_t*)(sp + s.off_pos);
    h->st.pbar = (float*)(sp + s.off_pbar);
    h->st.status = (int32_t*)(sp + s.off_status);
    uint8_t* cp = (uint8_t*)scratch;
    h->src = (int32_t*)cp;
    h->first_moved = (int32_t*)(cp + s.off_first);
    h->radix_list = (int32_t*)(cp + s.off_rlist);
    {
        const size_t qslot = align_up((size_t)h->layers * h->batch * h->q_heads * kRowBytes, 256);
        const size_t kslot = align_up((size_t)h->layers * h->batch * h->kv_heads * kRowBytes, 256);
        for (int i = 0; i < 2; ++i) {
            h->stage_q[i] = cp + s.off_q + i * qslot;
            h->stage_k[i] = cp + s.off_k + i * kslot;
            h->stage_v[i] = cp + s.off_v + i * kslot;
            h->stage_out[i] = cp + s.off_out + i * qslot;
        }
    }
    h->stage_score = (double*)(cp + s.off_score);
    h->stage_hist = (unsigned long long*)(cp + s.off_hist);
    h->h2_table = (double*)(cp + s.off_h2);
    h->h2_table_mode = -1;

    // Slots past n are read (and masked) by the decode kernel's last page: they must hold finite values.
    e = cudaMemsetAsync(h->pool, 0, s.kv, h->stream);
    if (e != cudaSuccess) return cuda_fail(h, e, "clearing the KV pool");
    e = init_state_launch(geometry(h), h->st, h->stream);
    if (e != cudaSuccess) return cuda_fail(h, e, "state initialisation launch");
    h->launches += 1;
    h->bound = true;
    return LAZYEV_OK;
}

int lazyev_set_page_table(lazyev_t* h, const int32_t* host_table) {
    if (!h) return LAZYEV_EINVAL;
    if (!h->bound || h->prefilled) return fail(h, LAZYEV_ESTATE, "set_page_table is only valid between bind and prefill");
    if (!host_table) return fail(h, LAZYEV_EINVAL, "null page table");
    const size_t total = (size_t)h->units * h->pages_per_unit;
    std::vector<char> seen(total, 0);
    for (size_t i = 0; i < total; ++i) {
        const int32_t p = host_table[i];
        if (p < 0 || (size_t)p >= total || seen[p]) return fail(h, LAZYEV_EINVAL, "page table is not a permutation");
        seen[p] = 1;
    }
    cudaError_t e = cudaMemcpyAsync(h->st.page_table, host_table, total * sizeof(int32_t), cudaMemcpyHostToDevice, h->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
    if (e != cudaSuccess) return cuda_fail(h, e, "page table upload");
    return LAZYEV_OK;
}

int lazyev_prefill(lazyev_t* h, const void* k, const void* v, int n_tokens) {
    if (!h) return LAZYEV_EINVAL;
    if (!h->bound) return fail(h, LAZYEV_ESTATE, "prefill before bind");
    if (h->prefilled) return fail(h, LAZYEV_ESTATE, "prefill called twice");
    if (!k || !v || n_tokens <= 0) return fail(h, LAZYEV_EINVAL, "null pointer or non-positive token count");
    if (n_tokens > h->max_prefill) return fail(h, LAZYEV_ECAPACITY, "prompt of %d tokens exceeds max_prefill = %d", n_tokens, h->max_prefill);
    cudaError_t e = prefill_launch(geometry(h), h->pool, h->st, k, v, n_tokens, INT_MIN, h->stream);
    if (e != cudaSuccess) return cuda_fail(h, e, "prefill kernel launch");
    h->launches += 1;
    h->prefilled = true;
    h->prefill = n_tokens;
    h->n = n_tokens;
    h->t = 0;
    return LAZYEV_OK;
}

namespace {
int host_wait(lazyev_t* h, int allowed);
}

int lazyev_reset(lazyev_t* h) {
    if (!h) return LAZYEV_EINVAL;
    if (!h->bound) return fail(h, LAZYEV_ESTATE, "reset before bind");
    if (h->copy_in) {                       // steps queued through the asynchronous host entry point finish first
        const int rc = host_wait(h, 0);
        if (rc != LAZYEV_OK) return rc;
    }
    // Old rows stay in the pool: slots past n are masked, they only have to be finite.  The state arrays
    // are rewritten by the next prompt load and by every append; the device status word is cleared.
    cudaError_t e = cudaMemsetAsync(h->st.status, 0, 64, h->stream);
    if (e != cudaSuccess) return cuda_fail(h, e, "clearing the device status word");
    h->prefilled = false;
    h->t = h->n = h->prefill = 0;
    h->budget_now = h->budget;
    return LAZYEV_OK;
}

int lazyev_prefill_observed(lazyev_t* h, const void* q, const void* k, const void* v, int n_tokens, void* out) {
    if (!h) return LAZYEV_EINVAL;
    if (!h->bound) return fail(h, LAZYEV_ESTATE, "prefill before bind");
    if (h->prefilled) return fail(h, LAZYEV_ESTATE, "prefill called twice");
    if (!q || !k || !v || !out || n_tokens <= 0) return fail(h, LAZYEV_EINVAL, "null pointer or non-positive token count");
    if (n_tokens > h->max_prefill) return fail(h, LAZYEV_ECAPACITY, "prompt of %d tokens exceeds max_prefill = %d", n_tokens, h->max_prefill);
    if (h->prompt_mode == LAZYEV_PROMPT_TILED && (((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out) & 15))
        return fail(h, LAZYEV_EINVAL, "q, k, v and out must be 16-byte aligned");
    // rows are loaded with TS = their own time j - (P - 1) <= 0 and MRI = 0
    cudaError_t e = prefill_launch(geometry(h), h->pool, h->st, k, v, n_tokens, 1 - n_tokens, h->stream);
    if (e != cudaSuccess) return cuda_fail(h, e, "prefill kernel launch");
    h->launches += 1;
    if (h->prompt_mode == LAZYEV_PROMPT_TILED) {
        // one launch: tiled causal attention on the tensor cores, K / V read once per query tile
        PromptArgs a;
        a.q = q;
        a.k = k;
        a.v = v;
        a.out = out;
        a.n_tokens = n_tokens;
        a.alpha = h->alpha;
        a.dump = h->prompt_dump;
        a.dump_begin = h->prompt_dump_begin;
        a.dump_count = h->prompt_dump_count;
        a.wait_limit_ns = h->wait_limit_ns;
        a.stop_after_tiles = h->stop_after_pages;
        e = prompt_launch(geometry(h), h->st, a, h->num_sms, h->stream);
        if (e != cudaSuccess) return cuda_fail(h, e, "prompt kernel launch");
        h->launches += 1;
    } else {
        // the prompt replayed through the decode kernel, one row per launch
        const size_t row_bytes = (size_t)h->layers * h->batch * h->q_heads * kRowBytes;
        for (int j = 0; j < n_tokens; ++j) {
            const int rc = run_decode(h, (const uint8_t*)q + j * row_bytes, (uint8_t*)out + j * row_bytes, j + 1,
                                      j - (n_tokens - 1), nullptr);
            if (rc != LAZYEV_OK) return rc;
            if (h->prompt_dump) {    // row j of the per-row probabilities: tokens 0 .. j of the dumped units
                e = cudaMemcpy2DAsync(h->prompt_dump + (size_t)j * n_tokens, (size_t)n_tokens * n_tokens * sizeof(float),
                                      h->st.pbar + (size_t)h->prompt_dump_begin * h->capacity, (size_t)h->capacity * sizeof(float),
                                      (size_t)(j + 1) * sizeof(float), h->prompt_dump_count, cudaMemcpyDeviceToDevice, h->stream);
                if (e != cudaSuccess) return cuda_fail(h, e, "prompt probability dump");
            }
        }
    }
    h->prefilled = true;
    h->prefill = n_tokens;
    h->n = n_tokens;
    h->t = 0;
    return LAZYEV_OK;
}

int lazyev_set_prompt_mode(lazyev_t* h, int mode) {
    if (!h) return LAZYEV_EINVAL;
    if (mode != LAZYEV_PROMPT_TILED && mode != LAZYEV_PROMPT_REPLAY) return fail(h, LAZYEV_EINVAL, "unknown prompt mode %d", mode);
    h->prompt_mode = mode;
    return LAZYEV_OK;
}

int lazyev_set_prompt_dump(lazyev_t* h, float* device_rows, int unit_begin, int unit_count) {
    if (!h) return LAZYEV_EINVAL;
    if (device_rows && (unit_begin < 0 || unit_count <= 0 || unit_begin + unit_count > h->units))
        return fail(h, LAZYEV_EINVAL, "unit range out of bounds");
    h->prompt_dump = device_rows;
    h->prompt_dump_begin = device_rows ? unit_begin : 0;
    h->prompt_dump_count = device_rows ? unit_count : 0;
    return LAZYEV_OK;
}

int lazyev_set_fused_append(lazyev_t* h, int on) {
    if (!h) return LAZYEV_EINVAL;
    h->fuse_append = on != 0;
    return LAZYEV_OK;
}

int lazyev_debug_starve_page_ring(lazyev_t* h, int pages) {
    if (!h) return LAZYEV_EINVAL;
    if (pages < -1) return fail(h, LAZYEV_EINVAL, "pages must be -1 (off) or >= 0");
    h->stop_after_pages = pages;
    return LAZYEV_OK;
}

int lazyev_set_wait_limit(lazyev_t* h, double seconds) {
    if (!h) return LAZYEV_EINVAL;
    if (!(seconds >= 1e-4 && seconds <= 60.0)) return fail(h, LAZYEV_EINVAL, "wait limit must be between 0.1 ms and 60 s");
    h->wait_limit_ns = (unsigned long long)(seconds * 1e9);
    return LAZYEV_OK;
}

int lazyev_decode_step(lazyev_t* h, const void* q, const void* k_new, const void* v_new, void* out) {
    if (!h) return LAZYEV_EINVAL;
    if (!q || !k_new || !v_new || !out) return fail(h, LAZYEV_EINVAL, "null pointer");
    return run_step(h, q, k_new, v_new, out);
}

namespace {

int host_streams(lazyev_t* h) {      // first host-buffer call: the two copy streams and their events
    if (h->copy_in) return LAZYEV_OK;
    cudaError_t e = cudaStreamCreateWithFlags(&h->copy_in, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&h->copy_out, cudaStreamNonBlocking);
    for (int i = 0; i <= kHostChunks && e == cudaSuccess; ++i) {
        e = cudaEventCreateWithFlags(&h->ev_in[i], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_done[i], cudaEventDisableTiming);
    }
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_ready, cudaEventDisableTiming);
    for (int i = 0; i < 2 && e == cudaSuccess; ++i)
        e = cudaEventCreateWithFlags(&h->ev_step_done[i], cudaEventDisableTiming | cudaEventBlockingSync);
    if (e != cudaSuccess) return cuda_fail(h, e, "creating the copy streams");
    return LAZYEV_OK;
}

// Blocks until at most `allowed` (0 or 1) asynchronous host-buffer steps are still in flight.
int host_wait(lazyev_t* h, int allowed) {
    cudaError_t e = cudaSuccess;
    const int newest = (int)((h->host_seq + 1) & 1);       // slot of the step queued last
    for (int k = 0; k < 2; ++k) {
        const int slot = k == 0 ? newest ^ 1 : newest;      // older step first
        if (!h->slot_busy[slot] || (allowed >= 1 && slot == newest)) continue;
        const cudaError_t e1 = cudaEventSynchronize(h->ev_step_done[slot]);
        if (e == cudaSuccess) e = e1;
        h->slot_busy[slot] = false;
    }
    if (e != cudaSuccess) return cuda_fail(h, e, "waiting for a host-buffer step");
    return LAZYEV_OK;
}

}  // namespace

int lazyev_decode_step_host(lazyev_t* h, const void* q, const void* k_new, const void* v_new, void* out) {
    if (!h) return LAZYEV_EINVAL;
    if (!q || !k_new || !v_new || !out) return fail(h, LAZYEV_EINVAL, "null pointer");
    if (!h->prefilled) return fail(h, LAZYEV_ESTATE, "decode_step before prefill");
    int rc = host_streams(h);
    if (rc == LAZYEV_OK) rc = host_wait(h, 0);
    if (rc != LAZYEV_OK) return rc;
    // The copy streams start after everything queued on the bound stream so far (an earlier step's
    // kernels may still read the staging buffers).
    cudaError_t e = cudaEventRecord(h->ev_ready, h->stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(h->copy_in, h->ev_ready, 0);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(h->copy_out, h->ev_ready, 0);
    const size_t kbytes = (size_t)h->layers * h->batch * h->kv_heads * kRowBytes;
    if (e == cudaSuccess) e = cudaMemcpyAsync(h->stage_k[0], k_new, kbytes, cudaMemcpyHostToDevice, h->stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h->stage_v[0], v_new, kbytes, cudaMemcpyHostToDevice, h->stream);
    if (e != cudaSuccess) return cuda_fail(h, e, "host-to-device copy");
    const HostPipe pipe{(const uint8_t*)q, (uint8_t*)out};
    rc = run_step(h, h->stage_q[0], h->stage_k[0], h->stage_v[0], h->stage_out[0], &pipe);
    // both streams are drained even after an error, so that no copy is left in flight on the caller's buffers
    cudaError_t e1 = cudaStreamSynchronize(h->copy_in), e2 = cudaStreamSynchronize(h->copy_out);
    e = cudaStreamSynchronize(h->stream);
    if (rc != LAZYEV_OK) return rc;
    if (e1 != cudaSuccess || e2 != cudaSuccess || e != cudaSuccess)
        return cuda_fail(h, e1 != cudaSuccess ? e1 : (e2 != cudaSuccess ? e2 : e), "copies of the host-buffer step");
    return LAZYEV_OK;
}

int lazyev_decode_step_host_async(lazyev_t* h, const void* q, const void* k_new, const void* v_new, void* out) {
    if (!h) return LAZYEV_EINVAL;
    if (!q || !k_new || !v_new || !out) return fail(h, LAZYEV_EINVAL, "null pointer");
    if (!h->prefilled) return fail(h, LAZYEV_ESTATE, "decode_step before prefill");
    int rc = host_streams(h);
    if (rc != LAZYEV_OK) return rc;
    const int slot = (int)(h->host_seq & 1);
    // The slot's previous step (two steps back) must be complete before its staging buffers are
    // reused; the step before this one may still be running, and this step's uploads run beside it.
    if (h->slot_busy[slot]) {
        const cudaError_t e0 = cudaEventSynchronize(h->ev_step_done[slot]);
        h->slot_busy[slot] = false;
        if (e0 != cudaSuccess) return cuda_fail(h, e0, "waiting for a host-buffer step");
    }
    const size_t qbytes = (size_t)h->layers * h->batch * h->q_heads * kRowBytes;
    const size_t kbytes = (size_t)h->layers * h->batch * h->kv_heads * kRowBytes;
    cudaError_t e = cudaSuccess;
    if (h->host_seq == 0 || !h->slot_busy[slot ^ 1]) {
        // nothing of ours in flight: order the copy streams after whatever else the bound stream holds
        e = cudaEventRecord(h->ev_ready, h->stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(h->copy_in, h->ev_ready, 0);
    }
    if (e == cudaSuccess) e = cudaMemcpyAsync(h->stage_k[slot], k_new, kbytes, cudaMemcpyHostToDevice, h->copy_in);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h->stage_v[slot], v_new, kbytes, cudaMemcpyHostToDevice, h->copy_in);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h->stage_q[slot], q, qbytes, cudaMemcpyHostToDevice, h->copy_in);
    if (e == cudaSuccess) e = cudaEventRecord(h->ev_in[0], h->copy_in);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(h->stream, h->ev_in[0], 0);
    if (e != cudaSuccess) return cuda_fail(h, e, "host-to-device copy");
    rc = run_step(h, h->stage_q[slot], h->stage_k[slot], h->stage_v[slot], h->stage_out[slot]);
    if (rc != LAZYEV_OK) return rc;      // found before anything was queued (see lazyev_decode_step)
    e = cudaEventRecord(h->ev_done[0], h->stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(h->copy_out, h->ev_done[0], 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(out, h->stage_out[slot], qbytes, cudaMemcpyDeviceToHost, h->copy_out);
    if (e == cudaSuccess) e = cudaEventRecord(h->ev_step_done[slot], h->copy_out);
    if (e != cudaSuccess) return cuda_fail(h, e, "device-to-host copy");
    h->slot_busy[slot] = true;
    h->host_seq += 1;
    return LAZYEV_OK;
}

int lazyev_host_wait(lazyev_t* h, int in_flight_allowed) {
    if (!h) return LAZYEV_EINVAL;
    if (in_flight_allowed < 0 || in_flight_allowed > 1) return fail(h, LAZYEV_EINVAL, "in_flight_allowed must be 0 or 1");
    if (!h->copy_in) return LAZYEV_OK;
    return host_wait(h, in_flight_allowed);
}

int lazyev_copy_state(lazyev_t* dst, lazyev_t* src) {
    if (!dst || !src || dst == src) return LAZYEV_EINVAL;
    if (!dst->bound || !src->bound) return fail(dst, LAZYEV_ESTATE, "copy_state needs two bound handles");
    if (!src->prefilled) return fail(dst, LAZYEV_ESTATE, "copy_state from a handle that holds no cache");
    if (dst->prefilled) return fail(dst, LAZYEV_ESTATE, "copy_state into a handle that already holds a cache (reset it first)");
    if (dst->device != src->device || dst->layers != src->layers || dst->batch != src->batch || dst->q_heads != src->q_heads ||
        dst->kv_heads != src->kv_heads || dst->capacity != src->capacity || dst->budget != src->budget ||
        dst->window != src->window || dst->n_recent != src->n_recent || dst->n_initial != src->n_initial)
        return fail(dst, LAZYEV_EINVAL, "copy_state needs two handles of the same configuration on the same device");
    const Sizes sz = sizes_of(src);
    cudaEvent_t ready = nullptr;
    cudaError_t e = cudaEventCreateWithFlags(&ready, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventRecord(ready, src->stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(dst->stream, ready, 0);
    // the state region starts with the page table, so the physical pages line up with the copied pool
    if (e == cudaSuccess) e = cudaMemcpyAsync(dst->pool, src->pool, sz.kv, cudaMemcpyDeviceToDevice, dst->stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dst->st.page_table, src->st.page_table, sz.state, cudaMemcpyDeviceToDevice, dst->stream);
    // and src's later steps must not overwrite what is still being read
    if (e == cudaSuccess) e = cudaEventRecord(ready, dst->stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(src->stream, ready, 0);
    if (ready) cudaEventDestroy(ready);
    if (e != cudaSuccess) return cuda_fail(dst, e, "copy_state");
    dst->prefilled = true;
    dst->t = src->t;
    dst->n = src->n;
    dst->prefill = src->prefill;
    dst->budget_now = src->budget_now;
    return LAZYEV_OK;
}

int lazyev_evict(lazyev_t* h, int* evicted) {
    if (!h) return LAZYEV_EINVAL;
    if (!h->prefilled) return fail(h, LAZYEV_ESTATE, "evict before prefill");
    return run_evict(h, evicted, h->src, h->first_moved, h->radix_list);
}

// ---- eviction without caller-provided scratch ------------------------------------------------
// Source lists and first-moved indices of lazyev_evict_static(): one array per GPU that loads the
// library, held until the process exits.  4 MiB + 32 KiB: source lists, first-moved indices, and the list
// of units that take the selection's general route.
constexpr size_t kStaticSrcEntries = (size_t)1 << 20;      // units * budget_now must not exceed this
constexpr int kStaticMaxUnits = 4096;
constexpr int kStaticMaxDevices = 64;
static __device__ __align__(256) int32_t g_static_evict_scratch[kStaticSrcEntries + 2 * kStaticMaxUnits + 64];
// Device addresses of the array above, one per device ordinal.  The symbol itself is only a
// host-side stand-in: kernels must be given the address cudaGetSymbolAddress() returns.
static std::atomic<int32_t*> g_static_evict_ptr[kStaticMaxDevices];

int lazyev_evict_static(lazyev_t* h, int* evicted) {
    if (!h) return LAZYEV_EINVAL;
    if (evicted) *evicted = 0;
    if (!h->prefilled) return fail(h, LAZYEV_ESTATE, "evict_static before prefill");
    if (h->units > kStaticMaxUnits || (size_t)h->units * (size_t)h->budget_now > kStaticSrcEntries)
        return fail(h, LAZYEV_ECAPACITY,
                    "evict_static holds %zu source indices for at most %d units; this handle needs %zu for %d units "
                    "(use lazyev_evict with the bound scratch region)",
                    kStaticSrcEntries, kStaticMaxUnits, (size_t)h->units * (size_t)h->budget_now, h->units);
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(h, e, "cudaGetDevice");
    if (dev != h->device || dev < 0 || dev >= kStaticMaxDevices)
        return fail(h, LAZYEV_ESTATE, "evict_static needs device %d (the one bound to this handle) to be current, not %d",
                    h->device, dev);
    int32_t* base = g_static_evict_ptr[dev].load(std::memory_order_acquire);
    if (!base) {    // first call on this device: resolve the array's device address (threads may race; same value)
        e = cudaGetSymbolAddress((void**)&base, g_static_evict_scratch);
        if (e != cudaSuccess || !base) return cuda_fail(h, e, "cudaGetSymbolAddress(static eviction scratch)");
        g_static_evict_ptr[dev].store(base, std::memory_order_release);
    }
    // Same trigger test, kernels, timing spans and accounting as lazyev_evict(); only the work lists
    // live elsewhere.  Every entry below budget is rewritten by the select kernel before the compact
    // kernel reads it, so nothing in the array has to be cleared.
    return run_evict(h, evicted, base, base + kStaticSrcEntries, base + kStaticSrcEntries + kStaticMaxUnits);
}

int lazyev_get_counters(lazyev_t* h, lazyev_counters_t* out) {
    if (!h || !out) return LAZYEV_EINVAL;
    if (!h->bound) return fail(h, LAZYEV_ESTATE, "get_counters before bind");
    int32_t words[16] = {0};
    cudaError_t e = cudaMemcpyAsync(words, h->st.status, sizeof(words), cudaMemcpyDeviceToHost, h->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
    if (e != cudaSuccess) return cuda_fail(h, e, "reading the device counters");
    out->device_status = words[0];
    out->select_radix_units = words[kCounterRadixUnits];
    out->select_zero_cut_units = words[kCounterZeroCutUnits];
    return LAZYEV_OK;
}

int lazyev_get_info(const lazyev_t* h, lazyev_info_t* out) {
    if (!h || !out) return LAZYEV_EINVAL;
    out->layers = h->layers;
    out->batch = h->batch;
    out->q_heads = h->q_heads;
    out->kv_heads = h->kv_heads;
    out->head_dim = h->head_dim;
    out->units = h->units;
    out->budget = h->budget;
    out->budget_now = h->budget_now;
    out->window = h->window;
    out->n_recent = h->n_recent;
    out->n_initial = h->n_initial;
    out->capacity = h->capacity;
    out->pages_per_unit = h->pages_per_unit;
    out->t = h->t;
    out->n = h->n;
    out->prefill = h->prefill;
    out->splits = h->last_plan.splits;
    out->stages = h->last_plan.stages;
    out->groups = h->last_plan.groups;
    out->tail_units = h->last_tail_units;
    out->tail_splits = h->last_tail_splits;
    out->grid = h->last_grid;
    out->smem_bytes = h->last_plan.smem_bytes;
    out->launches = h->launches;
    out->evictions = h->evictions;
    out->host_ranges = h->last_host_ranges;
    return LAZYEV_OK;
}

int lazyev_dump_state(lazyev_t* h, lazyev_dump_t* d) {
    if (!h || !d) return LAZYEV_EINVAL;
    if (!h->bound) return fail(h, LAZYEV_ESTATE, "dump before bind");
    if (d->unit_begin < 0 || d->unit_count < 0 || d->unit_begin + d->unit_count > h->units)
        return fail(h, LAZYEV_EINVAL, "unit range out of bounds");
    d->t = h->t;
    d->n = h->n;
    d->capacity = h->capacity;
    const size_t cap = h->capacity, first = (size_t)d->unit_begin * cap, count = (size_t)d->unit_count * cap;
    cudaError_t e = cudaSuccess;
    int32_t status = 0;
    e = cudaMemcpyAsync(&status, h->st.status, sizeof(status), cudaMemcpyDeviceToHost, h->stream);
    if (e == cudaSuccess && d->pos) e = cudaMemcpyAsync(d->pos, h->st.pos + first, count * 4, cudaMemcpyDeviceToHost, h->stream);
    std::vector<int2> pairs;               // TS and MRI sit interleaved on the device
    if (e == cudaSuccess && (d->ts || d->mri)) {
        pairs.resize(count);
        e = cudaMemcpyAsync(pairs.data(), h->st.tsm + first, count * sizeof(int2), cudaMemcpyDeviceToHost, h->stream);
    }
    if (e == cudaSuccess && d->pbar) e = cudaMemcpyAsync(d->pbar, h->st.pbar + first, count * 4, cudaMemcpyDeviceToHost, h->stream);
    if (e == cudaSuccess && !pairs.empty()) e = cudaStreamSynchronize(h->stream);
    if (e != cudaSuccess) return cuda_fail(h, e, "state download");
    for (size_t i = 0; i < pairs.size(); ++i) {
        if (d->ts) d->ts[i] = pairs[i].x;
        if (d->mri) d->mri[i] = pairs[i].y;
    }
    if (d->score) {
        const Geometry geo = geometry(h);
        for (int u0 = 0; u0 < d->unit_count; u0 += kScoreStageUnits) {
            const int cnt = d->unit_count - u0 < kScoreStageUnits ? d->unit_count - u0 : kScoreStageUnits;
            e = score_launch(geo, h->st, d->unit_begin + u0, cnt, h->n, h->t, h->score_mode, h->stage_score, h->stream);
            if (e == cudaSuccess)
                e = cudaMemcpyAsync(d->score + (size_t)u0 * cap, h->stage_score, (size_t)cnt * cap * sizeof(double), cudaMemcpyDeviceToHost, h->stream);
            if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
            if (e != cudaSuccess) return cuda_fail(h, e, "score download");
            h->launches += 1;
        }
    }
    if (d->k || d->v) {
        // Pages come back raw and are un-swizzled here on the host.
        const int np = (h->n + kPageTokens - 1) / kPageTokens;
        std::vector<int32_t> table((size_t)d->unit_count * h->pages_per_unit);
        e = cudaMemcpyAsync(table.data(), h->st.page_table + (size_t)d->unit_begin * h->pages_per_unit, table.size() * 4, cudaMemcpyDeviceToHost, h->stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
        if (e != cudaSuccess) return cuda_fail(h, e, "page table download");
        std::vector<uint8_t> page(kPageBytes);
        for (int u = 0; u < d->unit_count; ++u) {
            for (int pg = 0; pg < np; ++pg) {
                const int32_t pp = table[(size_t)u * h->pages_per_unit + pg];
                e = cudaMemcpyAsync(page.data(), h->pool + (size_t)pp * kPageBytes, kPageBytes, cudaMemcpyDeviceToHost, h->stream);
                if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
                if (e != cudaSuccess) return cuda_fail(h, e, "page download");
                for (int r = 0; r < kPageTokens; ++r) {
                    const size_t slot = (size_t)u * cap + (size_t)pg * kPageTokens + r;
                    for (int c = 0; c < kChunksPerRow; ++c) {
                        const uint8_t* ks = page.data() + r * kRowBytes + swz_chunk(c, r) * 16;
                        if (d->k) memcpy((uint8_t*)d->k + slot * kRowBytes + c * 16, ks, 16);
                        if (d->v) memcpy((uint8_t*)d->v + slot * kRowBytes + c * 16, ks + kPageHalfBytes, 16);
                    }
                }
            }
        }
    }
    e = cudaStreamSynchronize(h->stream);
    if (e != cudaSuccess) return cuda_fail(h, e, "stream synchronisation");
    d->device_status = status;
    if (status != 0) return fail(h, LAZYEV_EDEVICE, "device status word = %d (1: wait timed out, 2: bad index)", status);
    return LAZYEV_OK;
}

int lazyev_load_state(lazyev_t* h, const lazyev_dump_t* d, int prefill) {
    if (!h || !d) return LAZYEV_EINVAL;
    if (!h->bound) return fail(h, LAZYEV_ESTATE, "load_state before bind");
    if (h->prefilled) return fail(h, LAZYEV_ESTATE, "load_state on a handle that already holds a cache");
    if (d->unit_begin != 0 || d->unit_count != h->units) return fail(h, LAZYEV_EINVAL, "the snapshot must cover all %d units", h->units);
    if (!d->pos || !d->ts || !d->mri || !d->k || !d->v) return fail(h, LAZYEV_EINVAL, "pos, ts, mri, k and v are required");
    if (d->n <= 0 || d->n > h->capacity || d->capacity < d->n || d->t < 0 || prefill <= 0)
        return fail(h, LAZYEV_EINVAL, "snapshot sizes out of range (n = %d, capacity here = %d)", d->n, h->capacity);
    const size_t scap = (size_t)d->capacity, width = (size_t)d->n * 4;
    cudaError_t e = cudaMemcpy2DAsync(h->st.pos, (size_t)h->capacity * 4, d->pos, scap * 4, width, h->units, cudaMemcpyHostToDevice, h->stream);
    std::vector<int2> pairs((size_t)h->units * d->n);      // interleaved (TS, MRI), rows of n
    for (int u = 0; u < h->units; ++u)
        for (int i = 0; i < d->n; ++i)
            pairs[(size_t)u * d->n + i] = make_int2(d->ts[(size_t)u * scap + i], d->mri[(size_t)u * scap + i]);
    if (e == cudaSuccess)
        e = cudaMemcpy2DAsync(h->st.tsm, (size_t)h->capacity * 8, pairs.data(), (size_t)d->n * 8, (size_t)d->n * 8, h->units,
                              cudaMemcpyHostToDevice, h->stream);
    if (e == cudaSuccess && d->pbar) e = cudaMemcpy2DAsync(h->st.pbar, (size_t)h->capacity * 4, d->pbar, scap * 4, width, h->units, cudaMemcpyHostToDevice, h->stream);
    if (e != cudaSuccess) return cuda_fail(h, e, "state upload");
    // K / V rows: swizzled into pages on the host, one page per copy
    const int np = (d->n + kPageTokens - 1) / kPageTokens;
    std::vector<int32_t> table((size_t)h->units * h->pages_per_unit);
    e = cudaMemcpyAsync(table.data(), h->st.page_table, table.size() * 4, cudaMemcpyDeviceToHost, h->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
    if (e != cudaSuccess) return cuda_fail(h, e, "page table download");
    std::vector<uint8_t> page(kPageBytes);
    for (int u = 0; u < h->units; ++u) {
        for (int pg = 0; pg < np; ++pg) {
            memset(page.data(), 0, kPageBytes);
            for (int r = 0; r < kPageTokens && pg * kPageTokens + r < d->n; ++r) {
                const size_t slot = (size_t)u * scap + (size_t)pg * kPageTokens + r;
                for (int c = 0; c < kChunksPerRow; ++c) {
                    uint8_t* kd = page.data() + r * kRowBytes + swz_chunk(c, r) * 16;
                    memcpy(kd, (const uint8_t*)d->k + slot * kRowBytes + c * 16, 16);
                    memcpy(kd + kPageHalfBytes, (const uint8_t*)d->v + slot * kRowBytes + c * 16, 16);
                }
            }
            const int32_t pp = table[(size_t)u * h->pages_per_unit + pg];
            e = cudaMemcpyAsync(h->pool + (size_t)pp * kPageBytes, page.data(), kPageBytes, cudaMemcpyHostToDevice, h->stream);
            if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);      // the staging page is reused
            if (e != cudaSuccess) return cuda_fail(h, e, "page upload");
        }
    }
    h->prefilled = true;
    h->prefill = prefill;
    h->n = d->n;
    h->t = d->t;
    return LAZYEV_OK;
}

int lazyev_mri_histogram(lazyev_t* h, int unit_begin, int unit_count, long long* host_hist, int bins) {
    if (!h || !host_hist) return LAZYEV_EINVAL;
    if (!h->prefilled) return fail(h, LAZYEV_ESTATE, "mri_histogram before prefill");
    if (unit_begin < 0 || unit_count <= 0 || unit_begin + unit_count > h->units)
        return fail(h, LAZYEV_EINVAL, "unit range out of bounds");
    if (bins < 2 || bins > kMaxHistBins) return fail(h, LAZYEV_EINVAL, "bins must be in [2, %d]", kMaxHistBins);
    cudaError_t e = mri_histogram_launch(geometry(h), h->st, unit_begin, unit_count, h->n, bins, h->stage_hist, h->stream);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(host_hist, h->stage_hist, (size_t)bins * sizeof(long long), cudaMemcpyDeviceToHost, h->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
    if (e != cudaSuccess) return cuda_fail(h, e, "MRI histogram");
    h->launches += 1;
    return LAZYEV_OK;
}

int lazyev_mri_quantile(lazyev_t* h, int unit_begin, int unit_count, double fraction, int* value, long long* recurring) {
    if (!h || !value) return LAZYEV_EINVAL;
    if (!(fraction > 0.0 && fraction <= 1.0)) return fail(h, LAZYEV_EINVAL, "fraction must be in (0, 1]");
    std::vector<long long> hist(kMaxHistBins);
    const int rc = lazyev_mri_histogram(h, unit_begin, unit_count, hist.data(), kMaxHistBins);
    if (rc != LAZYEV_OK) return rc;
    long long total = 0;
    for (int b = 1; b < kMaxHistBins; ++b) total += hist[b];
    if (recurring) *recurring = total;
    *value = 0;
    if (total == 0) return LAZYEV_OK;
    // smallest v such that at least fraction * total of the re-activated tokens have MRI <= v
    long long cum = 0;
    for (int b = 1; b < kMaxHistBins; ++b) {
        cum += hist[b];
        if ((double)cum >= fraction * (double)total) {
            *value = b;
            break;
        }
    }
    return LAZYEV_OK;
}

int lazyev_set_profiling(lazyev_t* h, int on) {
    if (!h) return LAZYEV_EINVAL;
    if (!h->bound) return fail(h, LAZYEV_ESTATE, "set_profiling before bind");
    const int rc = collect_profile(h);
    h->profiling = on != 0;
    return rc;
}

int lazyev_get_profile(lazyev_t* h, lazyev_profile_t* out, int reset) {
    if (!h || !out) return LAZYEV_EINVAL;
    const int rc = collect_profile(h);
    if (rc != LAZYEV_OK) return rc;
    *out = h->prof;
    if (reset) h->prof = lazyev_profile_t{};
    return LAZYEV_OK;
}

int lazyev_synchronize(lazyev_t* h) {
    if (!h) return LAZYEV_EINVAL;
    if (!h->bound) return fail(h, LAZYEV_ESTATE, "synchronize before bind");
    if (h->copy_in) {
        const int rc = host_wait(h, 0);
        if (rc != LAZYEV_OK) return rc;
    }
    return check_device_status(h);
}

int lazyev_destroy(lazyev_t* h) {
    if (!h) return LAZYEV_EINVAL;
    if (h->copy_in) host_wait(h, 0);        // no copy of ours may still be writing the caller's host buffers
    for (const lazyev::Span& sp : h->pending) {
        cudaEventDestroy(sp.start);
        cudaEventDestroy(sp.stop);
    }
    for (cudaEvent_t e : h->free_events) cudaEventDestroy(e);
    if (h->tail_stream) cudaStreamDestroy(h->tail_stream);
    if (h->ev_fork) cudaEventDestroy(h->ev_fork);
    if (h->ev_join) cudaEventDestroy(h->ev_join);
    if (h->copy_in) cudaStreamDestroy(h->copy_in);
    if (h->copy_out) cudaStreamDestroy(h->copy_out);
    for (int i = 0; i <= kHostChunks; ++i) {
        if (h->ev_in[i]) cudaEventDestroy(h->ev_in[i]);
        if (h->ev_done[i]) cudaEventDestroy(h->ev_done[i]);
    }
    if (h->ev_ready) cudaEventDestroy(h->ev_ready);
    for (int i = 0; i < 2; ++i)
        if (h->ev_step_done[i]) cudaEventDestroy(h->ev_step_done[i]);
    delete h;
    return LAZYEV_OK;
}

}  // extern "C"
