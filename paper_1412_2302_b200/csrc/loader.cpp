// Host half of the paper's loading process ("Parallel Data Loading"): worker threads gather the next minibatches
// from a dataset in host memory (e.g. a memory-mapped uint8 file) into a ring of staging slots, in the order of a
// seeded per-epoch shuffle, while the consumer trains on the current one.  No CUDA calls: the ring is caller memory
// (pinned, if alexnet_load_batch_async is to copy from it asynchronously).
// All workers share every batch: a batch is cut into as many chunks of consecutive images as there are workers, handed
// out in order, so one batch is ready after batch / workers image copies per worker instead of `batch`; the copies
// bypass the cache on the store side (the ring is written once and next read by the GPU's copy engine), which
// saves the read-for-ownership of every destination line.
#include "../../include/alexnet.h"

#include <algorithm>
#include <chrono>
#include <condition_variable>
#include <cstring>
#include <mutex>
#include <thread>
#include <vector>
#if defined(__SSE2__)
#include <emmintrin.h>
#endif

namespace {
const size_t kImageBytes = 256 * 256 * 3;

// SplitMix64 finaliser as a counter hash (the same definition as the device kernels use, written out here again)
inline uint64_t mix64(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}
inline uint64_t draw(uint64_t key, uint64_t idx) { return mix64(key + 0x9E3779B97F4A7C15ULL * (idx + 1)); }

// copy with streaming (non-temporal) stores where the destination allows it
inline void copy_stream(uint8_t* dst, const uint8_t* src, size_t n) {
#if defined(__SSE2__)
    if (((uintptr_t)dst & 15) == 0) {
        size_t i = 0;
        for (; i + 64 <= n; i += 64) {
            const __m128i a = _mm_loadu_si128((const __m128i*)(src + i)), b = _mm_loadu_si128((const __m128i*)(src + i + 16));
            const __m128i c = _mm_loadu_si128((const __m128i*)(src + i + 32)), d = _mm_loadu_si128((const __m128i*)(src + i + 48));
            _mm_stream_si128((__m128i*)(dst + i), a); _mm_stream_si128((__m128i*)(dst + i + 16), b);
            _mm_stream_si128((__m128i*)(dst + i + 32), c); _mm_stream_si128((__m128i*)(dst + i + 48), d);
        }
        if (i < n) memcpy(dst + i, src + i, n - i);
        return;
    }
#endif
    memcpy(dst, src, n);
}
inline void store_fence() {
#if defined(__SSE2__)
    _mm_sfence();      // streaming stores become visible before the batch is published
#endif
}
}  // namespace

struct alexnet_loader {
    const uint8_t* images; const int32_t* labels;
    uint64_t n, n_epoch, seed; int batch, depth, shuffle, nthreads;
    uint8_t* ring; size_t slot_bytes;
    std::vector<std::thread> workers;
    std::mutex mu; std::condition_variable cv;
    // batch counters: released <= acquired <= released + depth; slot s holds batch ready[s] - 1 once filled
    uint64_t acquired = 0, released = 0;
    std::vector<uint64_t> ready;
    std::vector<int> chunks_done;     // per slot: chunks of the batch being filled that are finished
    uint64_t next_item = 0;           // work items are (batch, chunk) pairs in order: item = batch * nthreads + chunk
    bool stop = false;

    // the shuffle of one epoch: Fisher-Yates over the first n_epoch samples, draws from stream 9 keyed by the epoch
    void make_perm(std::vector<uint64_t>& perm, uint64_t epoch) const {
        perm.resize(n_epoch);
        for (uint64_t i = 0; i < n_epoch; ++i) perm[i] = i;
        if (shuffle) {
            const uint64_t key = mix64(seed ^ (9ULL << 56) ^ epoch);
            for (uint64_t i = n_epoch - 1; i > 0; --i) {
                const uint64_t j = draw(key, i) % (i + 1);
                std::swap(perm[i], perm[j]);
            }
        }
    }
    // Every worker takes the next (batch, chunk) item in order; chunk c of a batch is the images [c * batch / C, (c + 1) *
    // batch / C) with C = nthreads.  A slot may be refilled once the batch `depth` before has been released; the worker
    // that finishes the last chunk of a batch publishes it.
    void run() {
        std::vector<uint64_t> perm; uint64_t perm_epoch = ~0ULL;
        const uint64_t C = (uint64_t)nthreads;
        for (;;) {
            uint64_t b, c;
            {
                std::unique_lock<std::mutex> lk(mu);
                const uint64_t item = next_item++;
                b = item / C; c = item % C;
                cv.wait(lk, [&] { return stop || b < released + (uint64_t)depth; });
                if (stop) return;
            }
            uint8_t* slot = ring + (b % depth) * slot_bytes;
            int32_t* lab = (int32_t*)(slot + (size_t)batch * kImageBytes);
            const int i0 = (int)(c * (uint64_t)batch / C), i1 = (int)((c + 1) * (uint64_t)batch / C);
            for (int i = i0; i < i1; ++i) {
                const uint64_t j = b * (uint64_t)batch + i, epoch = j / n_epoch, pos = j % n_epoch;
                if (epoch != perm_epoch) { make_perm(perm, epoch); perm_epoch = epoch; }
                const uint64_t src = perm[pos];
                copy_stream(slot + (size_t)i * kImageBytes, images + src * kImageBytes, kImageBytes);
                lab[i] = labels[src];
            }
            store_fence();
            bool publish = false;
            {
                std::lock_guard<std::mutex> lk(mu);
                if (++chunks_done[b % depth] == (int)C) {
                    chunks_done[b % depth] = 0;
                    ready[b % depth] = b + 1;
                    publish = true;
                }
            }
            if (publish) cv.notify_all();
        }
    }
};

extern "C" {

size_t alexnet_loader_ring_bytes(int32_t batch, int32_t depth) {
    if (batch < 1 || depth < 2) return 0;
    const size_t slot = ((size_t)batch * kImageBytes + (size_t)batch * 4 + 4095) / 4096 * 4096;
    return slot * depth;
}

int alexnet_loader_create(const uint8_t* host_images, const int32_t* host_labels, uint64_t n_images, int32_t batch,
                          uint8_t* ring, size_t ring_bytes, int32_t depth, int32_t threads, uint64_t seed, int32_t shuffle,
                          alexnet_loader_t** out) {
    if (!out) return ALEXNET_ERR_ARG;
    *out = nullptr;
    if (!host_images || !host_labels || !ring || batch < 1 || depth < 2 || threads < 1 || threads > 64 || n_images < (uint64_t)batch)
        return ALEXNET_ERR_ARG;
    if (ring_bytes < alexnet_loader_ring_bytes(batch, depth)) return ALEXNET_ERR_NOMEM;
    alexnet_loader* l = new alexnet_loader();
    l->images = host_images; l->labels = host_labels; l->n = n_images; l->batch = batch; l->depth = depth;
    l->n_epoch = n_images / batch * batch;      // an epoch drops the incomplete last batch
    l->seed = seed; l->shuffle = shuffle ? 1 : 0;
    l->ring = ring; l->slot_bytes = alexnet_loader_ring_bytes(batch, depth) / depth;
    l->nthreads = std::min(threads, batch);      // a chunk holds at least one image
    l->ready.assign(depth, 0);
    l->chunks_done.assign(depth, 0);
    for (int t = 0; t < l->nthreads; ++t) l->workers.emplace_back([l] { l->run(); });
    *out = l;
    return ALEXNET_OK;
}

int alexnet_loader_next(alexnet_loader_t* l, int32_t timeout_ms, const uint8_t** images, const int32_t** labels, uint64_t* batch_index) {
    if (!l || !images || !labels) return ALEXNET_ERR_ARG;
    std::unique_lock<std::mutex> lk(l->mu);
    if (l->acquired >= l->released + (uint64_t)l->depth) return ALEXNET_ERR_STATE;      // every slot is held by the caller
    const uint64_t b = l->acquired;
    if (!l->cv.wait_for(lk, std::chrono::milliseconds(timeout_ms < 0 ? 0 : timeout_ms), [&] { return l->ready[b % l->depth] == b + 1; }))
        return ALEXNET_ERR_STATE;
    const uint8_t* slot = l->ring + (b % l->depth) * l->slot_bytes;
    *images = slot;
    *labels = (const int32_t*)(slot + (size_t)l->batch * kImageBytes);
    if (batch_index) *batch_index = b;
    l->acquired = b + 1;
    return ALEXNET_OK;
}

int alexnet_loader_release(alexnet_loader_t* l) {
    if (!l) return ALEXNET_ERR_ARG;
    {
        std::lock_guard<std::mutex> lk(l->mu);
        if (l->released >= l->acquired) return ALEXNET_ERR_STATE;
        l->released++;
    }
    l->cv.notify_all();
    return ALEXNET_OK;
}

int alexnet_loader_destroy(alexnet_loader_t* l) {
    if (!l) return ALEXNET_ERR_ARG;
    {
        std::lock_guard<std::mutex> lk(l->mu);
        l->stop = true;
    }
    l->cv.notify_all();
    for (std::thread& w : l->workers)
        if (w.joinable()) w.join();
    delete l;
    return ALEXNET_OK;
}

}  // extern "C"
