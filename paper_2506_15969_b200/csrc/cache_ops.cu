// Cache maintenance kernels: state initialisation, prompt load, per-step append.
#include <limits.h>

#include "internal.h"

namespace lzk {

namespace {

__global__ void init_state_kernel(Geometry geo, StateView st) {
    const size_t total_pages = (size_t)geo.units * geo.pages_per_unit;
    const size_t total_slots = (size_t)geo.units * geo.capacity;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total_slots; i += stride) {
        if (i < total_pages) st.page_table[i] = (int32_t)i;      // identity: unit u owns pages [u*ppu, (u+1)*ppu)
        if (i < 16) st.status[i] = 0;
        st.tsm[i] = make_int2(0, 0);
        st.pos[i] = 0;
        st.pbar[i] = 0.f;
    }
}

// One warp per (unit, token): lanes 0..15 move the K row's chunks, lanes 16..31 the V row's.
__global__ void prefill_kernel(Geometry geo, uint8_t* pool, StateView st, const uint4* __restrict__ k,
                               const uint4* __restrict__ v, int n_tokens, int ts_first) {
    const int lane = threadIdx.x & 31;
    const size_t warps = ((size_t)gridDim.x * blockDim.x) >> 5;
    const size_t total = (size_t)geo.units * n_tokens;
    for (size_t w = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; w < total; w += warps) {
        const int u = (int)(w / n_tokens), i = (int)(w % n_tokens);
        if (!in_bounds(i < geo.capacity, st.status)) continue;
        const int32_t pp = st.page_table[(size_t)u * geo.pages_per_unit + i / kPageTokens];
        if (!in_bounds(pp >= 0 && pp < geo.units * geo.pages_per_unit, st.status)) continue;
        const int r = i % kPageTokens, c = lane & 15;
        const uint4* src = (lane < 16 ? k : v) + w * kChunksPerRow + c;
        uint8_t* row = page_ptr(pool, pp) + (lane < 16 ? 0 : kPageHalfBytes) + r * kRowBytes;
        *reinterpret_cast<uint4*>(row + swz_chunk(c, r) * 16) = *src;
        if (lane == 0) {
            const size_t s = (size_t)u * geo.capacity + i;
            // Prompt tokens start at MRI = 0 (Section 4) and TS = 0, or, when the prompt is going to be
            // replayed with tracking, at their own time ts_first + i (the last prompt row is time 0).
            st.tsm[s] = make_int2(ts_first == INT_MIN ? 0 : ts_first + i, 0);
            st.pos[s] = i;
        }
    }
}

// One warp per unit: writes the new token's K / V rows into slot `slot`.
__global__ void append_kernel(Geometry geo, uint8_t* pool, StateView st, const uint4* __restrict__ k_new,
                              const uint4* __restrict__ v_new, int slot, int t, int position) {
    const int lane = threadIdx.x & 31;
    const int u = (int)(((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
    if (u >= geo.units) return;
    if (!in_bounds(slot >= 0 && slot < geo.capacity, st.status)) return;
    const int32_t pp = st.page_table[(size_t)u * geo.pages_per_unit + slot / kPageTokens];
    if (!in_bounds(pp >= 0 && pp < geo.units * geo.pages_per_unit, st.status)) return;
    const int r = slot % kPageTokens, c = lane & 15;
    const uint4* src = (lane < 16 ? k_new : v_new) + (size_t)u * kChunksPerRow + c;
    uint8_t* row = page_ptr(pool, pp) + (lane < 16 ? 0 : kPageHalfBytes) + r * kRowBytes;
    *reinterpret_cast<uint4*>(row + swz_chunk(c, r) * 16) = *src;
    if (lane == 0) {
        const size_t s = (size_t)u * geo.capacity + slot;
        st.tsm[s] = make_int2(t, 0);      // a token is born active at its own step, with MRI = 0
        st.pos[s] = position;
    }
}

}  // namespace

cudaError_t init_state_launch(const Geometry& geo, StateView st, cudaStream_t stream) {
    init_state_kernel<<<1184, 256, 0, stream>>>(geo, st);
    return cudaGetLastError();
}

cudaError_t prefill_launch(const Geometry& geo, uint8_t* pool, StateView st, const void* k, const void* v,
                           int n_tokens, int ts_first, cudaStream_t stream) {
    const size_t rows = (size_t)geo.units * n_tokens;
    const int blocks = (int)((rows + 7) / 8 < 148 * 16 ? (rows + 7) / 8 : 148 * 16);
    prefill_kernel<<<blocks, 256, 0, stream>>>(geo, pool, st, reinterpret_cast<const uint4*>(k),
                                               reinterpret_cast<const uint4*>(v), n_tokens, ts_first);
    return cudaGetLastError();
}

cudaError_t append_launch(const Geometry& geo, uint8_t* pool, StateView st, const void* k_new, const void* v_new,
                          int slot, int t, int position, cudaStream_t stream) {
    const int blocks = (geo.units + 7) / 8;
    append_kernel<<<blocks, 256, 0, stream>>>(geo, pool, st, reinterpret_cast<const uint4*>(k_new),
                                              reinterpret_cast<const uint4*>(v_new), slot, t, position);
    return cudaGetLastError();
}

}  // namespace lzk
