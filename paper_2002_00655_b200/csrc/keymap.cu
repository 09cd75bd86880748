// The sparse-map front end of the store (Section 3.7 of the paper: a server keeps its local parameters "in dense
// arrays or sparse maps").  Arbitrary 64-bit keys are translated to the dense keys 0 .. capacity-1 that the store's
// calls take; a key gets the next unused dense key the first time it is seen, in order of first appearance in the
// call, so a sequential program reproduces the translation exactly.
//
// The map is an open-addressing hash table in device memory (linear probing, at most half full).  An insert call
// is ONE cooperative launch:
//   1. every occurrence finds or claims its key's slot (compare-and-swap on the key word); an occurrence of a key
//      that is new in this call leaves its position in the slot's value word by atomic minimum, so that afterwards
//      the word names the key's first occurrence (values of keys inserted by earlier calls are smaller than any such
//      mark and are left alone)
//   2. first occurrences of new keys are counted per block                                   -> grid barrier
//   3. every block adds up the counts: its offset among the new keys, and their total; a call that would exceed the
//      capacity empties the slots it claimed (they were empty before the call, and only this call's keys can have
//      probed past them) and fails as a whole; otherwise first occurrences write their dense key  -> grid barrier
//   4. every occurrence reads its dense key from its slot.
#include <new>
#include <string.h>

#include "ps_internal.cuh"

struct ps_keymap {
    uint64_t capacity, n_slots, max_batch;
    int device, sm_count;
    unsigned long long* keys;           // n_slots; all ones = empty
    unsigned int* vals;                 // n_slots; dense key, or 0x80000000 | position of the first occurrence in the running call
    unsigned long long* size;           // dense keys handed out so far
    unsigned int* status;               // sticky error code
    unsigned int* bar;                  // two words of the grid barrier
    unsigned int* block_counts;         // 512
    unsigned int* slot_of;              // max_batch: the slot of every occurrence of the running call
    uint64_t launches;
};

namespace psb {

constexpr unsigned long long kEmptyKey = ~0ull;
constexpr uint32_t kMapMaxGrid = 2048;

__device__ __forceinline__ uint64_t mix64(uint64_t x) {         // an avalanche of xor-shifts and odd multiplications
    x ^= x >> 31;
    x *= 0x7fb5d329728ea185ull;
    x ^= x >> 27;
    x *= 0x81dadef4bc2dd44dull;
    x ^= x >> 33;
    return x;
}

static size_t pad256(size_t x) { return (x + 255) / 256 * 256; }

struct MapLayout {
    size_t keys, vals, size, status, bar, block_counts, slot_of, total;
    uint64_t n_slots;
};
static MapLayout map_layout(uint64_t capacity, uint64_t max_batch) {
    MapLayout l;
    uint64_t slots = 64;
    while (slots < 2 * capacity) slots <<= 1;
    l.n_slots = slots;
    size_t off = 0;
    auto take = [&](size_t b) { const size_t at = off; off = pad256(off + b); return at; };
    l.keys = take(slots * 8);
    l.vals = take(slots * 4);
    l.size = take(8);
    l.status = take(4);
    l.bar = take(8);
    l.block_counts = take(kMapMaxGrid * 4);
    l.slot_of = take((max_batch ? max_batch : 1) * 4);
    l.total = off;
    return l;
}

__global__ void map_clear_kernel(unsigned long long* keys, unsigned int* vals, uint64_t n_slots, unsigned long long* size,
                                 unsigned int* status, unsigned int* bar) {
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_slots; i += stride) {
        keys[i] = kEmptyKey;
        vals[i] = 0xFFFFFFFFu;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        *size = 0ull;
        *status = 0u;
        bar[0] = bar[1] = 0u;
    }
}

__global__ void __launch_bounds__(256)
map_insert_kernel(ps_keymap m, const uint64_t* __restrict__ in, uint32_t n, uint32_t span, uint64_t* __restrict__ out) {
    __shared__ uint32_t sm[8];
    __shared__ int s_ok;
    const int tid = threadIdx.x;
    const uint32_t b = blockIdx.x, G = gridDim.x;
    const uint32_t lo = (uint32_t)tmin<uint64_t>((uint64_t)b * span, n), hi = (uint32_t)tmin<uint64_t>((uint64_t)lo + span, n);
    const uint64_t mask = m.n_slots - 1;
    // ---- 1: find or claim the slot of every occurrence ----
    for (uint32_t t = lo + tid; t < hi; t += 256) {
        const unsigned long long key = in[t];
        uint64_t s = mix64(key) & mask;
        uint32_t found = 0xFFFFFFFFu;
        if (key != kEmptyKey) {                                 // (the all-ones key is the empty mark: refused below)
            for (uint64_t probes = 0; probes < m.n_slots; ++probes) {
                unsigned long long cur = __ldcg(&m.keys[s]);
                if (cur == kEmptyKey) cur = atomicCAS(&m.keys[s], kEmptyKey, key);
                if (cur == kEmptyKey || cur == key) {
                    found = (uint32_t)s;
                    break;
                }
                s = (s + 1) & mask;
            }
        }
        m.slot_of[t] = found;
        if (found == 0xFFFFFFFFu) atomicCAS(m.status, 0u, (unsigned int)PS_ERR_KEY_RANGE);
        else atomicMin(&m.vals[found], 0x80000000u | t);         // a dense key from an earlier call is smaller and stays
    }
    if (!grid_barrier(m.bar, G, &s_ok)) {
        if (tid == 0) atomicCAS(m.status, 0u, (unsigned int)PS_ERR_CUDA);
        return;
    }
    // ---- 2: first occurrences of new keys, per block ----
    const bool bad_key = *((volatile unsigned int*)m.status) == PS_ERR_KEY_RANGE;
    auto is_first = [&](uint32_t t) { return t < hi && m.slot_of[t] != 0xFFFFFFFFu && __ldcg(&m.vals[m.slot_of[t]]) == (0x80000000u | t); };
    uint32_t cnt = 0;
    for (uint32_t t0 = lo; t0 < hi; t0 += 256) cnt += (uint32_t)__syncthreads_count(is_first(t0 + tid));
    if (tid == 0) m.block_counts[b] = cnt;
    if (!grid_barrier(m.bar, 2 * G, &s_ok)) {
        if (tid == 0) atomicCAS(m.status, 0u, (unsigned int)PS_ERR_CUDA);
        return;
    }
    // ---- 3: dense keys for the new keys, or the whole call undone ----
    uint32_t before = 0, all = 0;
    for (uint32_t i = tid; i < G; i += 256) {
        const uint32_t v = __ldcg(m.block_counts + i);
        all += v;
        if (i < b) before += v;
    }
    uint32_t m0, total;
    block_exclusive_scan_256(before, sm, &m0);
    block_exclusive_scan_256(all, sm, &total);
    const unsigned long long size0 = *((volatile unsigned long long*)m.size);    // (rewritten only after the last barrier)
    const bool full = size0 + total > m.capacity;
    if (full && b == 0 && tid == 0) atomicCAS(m.status, 0u, (unsigned int)PS_ERR_CAPACITY);
    uint32_t running = 0;
    for (uint32_t t0 = lo; t0 < hi; t0 += 256) {
        const uint32_t t = t0 + tid;
        const bool f = is_first(t);
        uint32_t tot;
        const uint32_t ex = block_exclusive_scan_256(f ? 1u : 0u, sm, &tot);
        if (f) {
            const uint32_t s = m.slot_of[t];
            if (full || bad_key) {                              // give the slot back: it was empty before the call
                m.vals[s] = 0xFFFFFFFFu;
                m.keys[s] = kEmptyKey;
            } else {
                m.vals[s] = (uint32_t)(size0 + m0 + running + ex);
            }
        }
        running += tot;
    }
    if (!grid_barrier(m.bar, 3 * G, &s_ok)) {
        if (tid == 0) atomicCAS(m.status, 0u, (unsigned int)PS_ERR_CUDA);
        return;
    }
    // ---- 4: every occurrence reads its dense key ----
    for (uint32_t t = lo + tid; t < hi; t += 256) {
        const uint32_t s = m.slot_of[t];
        out[t] = (full || bad_key || s == 0xFFFFFFFFu) ? ~0ull : (uint64_t)__ldcg(&m.vals[s]);
    }
    if (b == 0 && tid == 0 && !full && !bad_key) *m.size = size0 + total;
    grid_leave(m.bar, G);
}

__global__ void __launch_bounds__(256)
map_lookup_kernel(ps_keymap m, const uint64_t* __restrict__ in, uint64_t n, uint64_t* __restrict__ out) {
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n) return;
    const unsigned long long key = in[t];
    const uint64_t mask = m.n_slots - 1;
    uint64_t s = mix64(key) & mask;
    uint64_t res = ~0ull;
    if (key != kEmptyKey) {
        for (uint64_t probes = 0; probes < m.n_slots; ++probes) {
            const unsigned long long cur = m.keys[s];
            if (cur == key) {
                res = m.vals[s];
                break;
            }
            if (cur == kEmptyKey) break;
            s = (s + 1) & mask;
        }
    }
    out[t] = res;
}

}  // namespace psb

using namespace psb;

extern "C" {

ps_status_t ps_keymap_query_bytes(uint64_t capacity, uint64_t max_batch_keys, size_t* out) {
    if (!out || capacity == 0 || capacity >= (1ull << 30) || max_batch_keys == 0 || max_batch_keys >= (1ull << 31))
        return PS_ERR_INVALID_ARG;
    *out = map_layout(capacity, max_batch_keys).total;
    return PS_OK;
}

ps_status_t ps_keymap_create(uint64_t capacity, uint64_t max_batch_keys, void* d_mem, size_t bytes, int32_t device,
                             void* stream, ps_keymap_t** out) {
    size_t need = 0;
    if (!out || !d_mem || ((uintptr_t)d_mem & 255)) return PS_ERR_INVALID_ARG;
    const ps_status_t c = ps_keymap_query_bytes(capacity, max_batch_keys, &need);
    if (c != PS_OK) return c;
    if (bytes < need) return PS_ERR_WORKSPACE;
    if (cudaSetDevice(device) != cudaSuccess) return PS_ERR_CUDA;
    ps_keymap* m = new (std::nothrow) ps_keymap();
    if (!m) return PS_ERR_INVALID_ARG;
    memset(m, 0, sizeof *m);
    const MapLayout l = map_layout(capacity, max_batch_keys);
    char* base = (char*)d_mem;
    m->capacity = capacity;
    m->n_slots = l.n_slots;
    m->max_batch = max_batch_keys;
    m->device = device;
    m->keys = (unsigned long long*)(base + l.keys);
    m->vals = (unsigned int*)(base + l.vals);
    m->size = (unsigned long long*)(base + l.size);
    m->status = (unsigned int*)(base + l.status);
    m->bar = (unsigned int*)(base + l.bar);
    m->block_counts = (unsigned int*)(base + l.block_counts);
    m->slot_of = (unsigned int*)(base + l.slot_of);
    if (cudaDeviceGetAttribute(&m->sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || m->sm_count <= 0) {
        delete m;
        return PS_ERR_CUDA;
    }
    const uint32_t grid = (uint32_t)tmin<uint64_t>((l.n_slots + 255) / 256, (uint64_t)m->sm_count * 16);
    map_clear_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>(m->keys, m->vals, m->n_slots, m->size, m->status, m->bar);
    m->launches = 1;
    if (cudaGetLastError() != cudaSuccess) {
        delete m;
        return PS_ERR_CUDA;
    }
    *out = m;
    return PS_OK;
}

ps_status_t ps_keymap_destroy(ps_keymap_t* m) {
    if (!m) return PS_ERR_INVALID_ARG;
    cudaSetDevice(m->device);
    cudaDeviceSynchronize();
    delete m;
    return PS_OK;
}

ps_status_t ps_keymap_insert(ps_keymap_t* m, const uint64_t* d_sparse, uint64_t n, uint64_t* d_dense, void* stream) {
    if (!m) return PS_ERR_INVALID_ARG;
    if (n == 0) return PS_OK;
    if (!d_sparse || !d_dense) return PS_ERR_INVALID_ARG;
    if (n > m->max_batch) return PS_ERR_WORKSPACE;
    // All blocks are resident at once (they meet at grid barriers).  The probes are chains of dependent random reads,
    // so the kernel wants as many threads in flight as fit: eight blocks per SM (the kernel is light on registers).
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, (const void*)map_insert_kernel, 256, 0) != cudaSuccess || per_sm < 1)
        return PS_ERR_CUDA;
    const uint32_t max_grid = tmin<uint32_t>((uint32_t)m->sm_count * (uint32_t)tmin(per_sm, 8), kMapMaxGrid);
    uint32_t n32 = (uint32_t)n;
    uint32_t span = tmax<uint32_t>(div_up_u32(n, max_grid), 256u);
    const uint32_t grid = div_up_u32(n, span);
    ps_keymap km = *m;
    void* args[] = {(void*)&km, (void*)&d_sparse, (void*)&n32, (void*)&span, (void*)&d_dense};
    cudaLaunchCooperativeKernel((const void*)map_insert_kernel, dim3(grid), dim3(256), args, 0, (cudaStream_t)stream);
    m->launches++;
    return cudaGetLastError() == cudaSuccess ? PS_OK : PS_ERR_CUDA;
}

ps_status_t ps_keymap_lookup(ps_keymap_t* m, const uint64_t* d_sparse, uint64_t n, uint64_t* d_dense, void* stream) {
    if (!m) return PS_ERR_INVALID_ARG;
    if (n == 0) return PS_OK;
    if (!d_sparse || !d_dense) return PS_ERR_INVALID_ARG;
    map_lookup_kernel<<<div_up_u32(n, 256), 256, 0, (cudaStream_t)stream>>>(*m, d_sparse, n, d_dense);
    m->launches++;
    return cudaGetLastError() == cudaSuccess ? PS_OK : PS_ERR_CUDA;
}

ps_status_t ps_keymap_sync(ps_keymap_t* m, void* stream, uint64_t* h_size) {
    if (!m) return PS_ERR_INVALID_ARG;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return PS_ERR_CUDA;
    unsigned int code = 0;
    unsigned long long size = 0;
    if (cudaMemcpy(&code, m->status, 4, cudaMemcpyDeviceToHost) != cudaSuccess ||
        cudaMemcpy(&size, m->size, 8, cudaMemcpyDeviceToHost) != cudaSuccess)
        return PS_ERR_CUDA;
    if (code != 0) {
        if (cudaMemset(m->status, 0, 4) != cudaSuccess) return PS_ERR_CUDA;
        if (code == PS_ERR_CUDA && cudaMemset(m->bar, 0, 8) != cudaSuccess) return PS_ERR_CUDA;   // a barrier that gave up
    }
    if (h_size) *h_size = size;
    return (ps_status_t)code;
}

uint64_t ps_keymap_launch_count(const ps_keymap_t* m) { return m ? m->launches : 0; }

}  // extern "C"
