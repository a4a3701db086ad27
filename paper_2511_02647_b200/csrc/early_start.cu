// Host-side bookkeeping for kernels that are launched with programmatic stream serialization and
// read their inputs, or write their outputs, before they wait for the preceding grid of the stream.
//
// Such a kernel releases its own dependents when it starts and calls griddepcontrol.wait later (at the
// latest in one closing CTA, so that a grid never completes before its predecessor).  Reading early is
// sound as long as nothing that may still be running writes the inputs; writing early is sound as long
// as nothing that may still be running reads or writes the outputs.  The only grids that release
// dependents early are this library's own (every other kernel of the stream is taken to be launched
// without the programmatic attribute, or to wait before it ends), so the only accesses that can still
// be in flight are those of recent library calls of that kind.  Grids of this kind can pile up (each
// only needs its predecessor to have STARTED), so the record keeps every buffer such a call reads or
// writes since the last call of the stream that waited first.
//
//   * A call whose inputs overlap a recorded WRITE waits first (griddepcontrol.wait, then release):
//     its successors then start only when everything before them is complete, which empties the
//     record (the call's own buffers are recorded afresh).
//   * A call that writes before it waits must know that every recorded reader and writer of its
//     outputs is over.  Calls of one context carry sequence numbers, and the context keeps a device
//     word `done` = the largest sequence number whose call is known to be complete (written by a
//     later call's closing CTA after ITS griddepcontrol.wait returned).  The launcher hands the kernel
//     the number it needs (`need_seq`); the kernel writes at once when done >= need_seq and waits for
//     the preceding grid otherwise.  An overlap with a call that has no sequence number in that
//     context (another kind of call, another context) makes the whole call wait first.
//   * Records are kept per stream: ordering between streams is the caller's (events complete a grid
//     before they fire).  A stream without a record (never seen, or displaced by others) waits first.
//     When a context moves to another stream its sequence numbers lose their meaning there: its
//     entries become anonymous.
//   * While a stream is being captured the calls are recorded under the capture's own key, carry no
//     sequence number and publish nothing: the values baked into a captured launch must hold for every
//     replay, so a captured call whose outputs overlap an earlier captured call's buffers always waits
//     before it writes (need_seq = INT64_MAX) but may still read early.
#include <memory>
#include <mutex>

#include "common.cuh"

namespace fedattn {

namespace {

constexpr int kRecord = 320;       // ranges per stream; one call has at most 2 * kMaxP + 5
constexpr int kSlots = 8;          // streams (or captures) remembered per device
struct Slot {
    uint64_t key = 0, last_use = 0;
    int n = 0;
    uintptr_t lo[kRecord], hi[kRecord];
    const void *owner[kRecord];    // whose sequence numbers `seq` counts in (a context's done word), or null
    int64_t seq[kRecord];          // the owner's latest call that touches this range
    uint8_t rd[kRecord];           // 1: read by that call, 0: written
};
struct DeviceRecord {
    Slot slot[kSlots];
    int n_slots = 0;
    uint64_t clock = 0;
};
std::unique_ptr<DeviceRecord> g_record[64];
std::mutex g_record_mutex;

struct Range {
    uintptr_t lo, hi;
    uint8_t rd;
};

}  // namespace

EarlyStart early_start(int device, cudaStream_t stream, const MemRange *in, int n_in, const MemRange *out, int n_out,
                       bool writes_before_wait, const void *owner, int64_t *seq_counter, uint64_t *owner_key)
{
    EarlyStart r{false, 0, 0};
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    unsigned long long cap_id = 0;
    if (cudaStreamGetCaptureInfo(stream, &cap, &cap_id) != cudaSuccess) {
        cudaGetLastError();
        cap = cudaStreamCaptureStatusNone;
    }
    const bool capturing = cap != cudaStreamCaptureStatusNone;
    const uint64_t key = capturing ? (((uint64_t)(uintptr_t)stream * 0x9E3779B97F4A7C15ull) ^ (cap_id << 1)) | 1ull
                                   : (uint64_t)(uintptr_t)stream << 1;
    if (capturing) owner = nullptr;

    std::lock_guard<std::mutex> lock(g_record_mutex);
    std::unique_ptr<DeviceRecord> &dev = g_record[device & 63];
    if (!dev) dev.reset(new DeviceRecord);
    bool wait_first = false;
    Slot *sl = nullptr;
    for (int i = 0; i < dev->n_slots; ++i)
        if (dev->slot[i].key == key) sl = &dev->slot[i];
    if (!sl) {                                                    // nothing is known about this stream
        if (dev->n_slots < kSlots) sl = &dev->slot[dev->n_slots++];
        else {
            sl = &dev->slot[0];
            for (int i = 1; i < kSlots; ++i)
                if (dev->slot[i].last_use < sl->last_use) sl = &dev->slot[i];
        }
        sl->key = key;
        sl->n = 0;
        wait_first = true;
    }
    sl->last_use = ++dev->clock;
    if (owner && owner_key && *owner_key != key) {                // the context has moved to this stream
        for (int i = 0; i < dev->n_slots; ++i)
            for (int j = 0; j < dev->slot[i].n; ++j)
                if (dev->slot[i].owner[j] == owner) dev->slot[i].owner[j] = nullptr;
        *owner_key = key;
    }
    const int64_t seq = (owner && seq_counter) ? ++*seq_counter : 0;
    r.seq = seq;

    Range mine[2 * kMaxP + 24];
    int n_mine = 0;
    bool too_many = false;
    auto add = [&](const MemRange &m, uint8_t rd) {
        if (!m.p || !m.bytes) return;
        if (n_mine == (int)(sizeof(mine) / sizeof(mine[0]))) { too_many = true; return; }
        const uintptr_t lo = reinterpret_cast<uintptr_t>(m.p);
        mine[n_mine++] = Range{lo, lo + m.bytes, rd};
    };
    for (int i = 0; i < n_in; ++i) add(in[i], 1);
    for (int o = 0; o < n_out; ++o) add(out[o], 0);
    if (too_many || n_mine > kRecord) {
        // cannot be recorded: wait first, and leave one entry that makes the next call wait first too
        sl->n = 1;
        sl->lo[0] = 0; sl->hi[0] = UINTPTR_MAX; sl->owner[0] = nullptr; sl->seq[0] = 0; sl->rd[0] = 0;
        return r;
    }

    int64_t need = 0;
    bool unknown = false;
    int match[2 * kMaxP + 24];
    int n_new = 0;
    for (int i = 0; i < n_mine; ++i) {
        const Range &m = mine[i];
        match[i] = -1;
        for (int j = 0; j < sl->n; ++j) {
            if (!(m.lo < sl->hi[j] && sl->lo[j] < m.hi)) continue;
            if (m.rd) {
                if (!sl->rd[j]) wait_first = true;                // an input that may still be being written
            } else if (writes_before_wait) {
                if (owner && sl->owner[j] == owner) need = need > sl->seq[j] ? need : sl->seq[j];
                else unknown = true;                              // a reader or writer that cannot be named
            }
            if (m.lo == sl->lo[j] && m.hi == sl->hi[j] && m.rd == sl->rd[j] && sl->owner[j] == owner) match[i] = j;
        }
        n_new += match[i] < 0;
    }
    if (unknown) {
        if (capturing) need = INT64_MAX;
        else wait_first = true;
    }
    if (sl->n + n_new > kRecord) wait_first = true;
    if (wait_first) {                                             // nothing before this call is left when it runs
        sl->n = 0;
        need = 0;
    }
    for (int i = 0; i < n_mine; ++i) {
        int j = wait_first ? -1 : match[i];
        if (j < 0) j = sl->n++;
        sl->lo[j] = mine[i].lo; sl->hi[j] = mine[i].hi; sl->rd[j] = mine[i].rd;
        sl->owner[j] = owner; sl->seq[j] = seq;
    }
    r.early = !wait_first;
    r.need_seq = need;
    return r;
}

void early_start_forget(int device, const void *owner)
{
    std::lock_guard<std::mutex> lock(g_record_mutex);
    DeviceRecord *dev = g_record[device & 63].get();
    if (!dev || !owner) return;
    for (int i = 0; i < dev->n_slots; ++i)
        for (int j = 0; j < dev->slot[i].n; ++j)
            if (dev->slot[i].owner[j] == owner) dev->slot[i].owner[j] = nullptr;
}

}  // namespace fedattn
