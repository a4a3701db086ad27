// Host-side bookkeeping for kernels that are launched with programmatic stream serialization and
// read their inputs before they wait for the preceding grid of the stream.
//
// Such a kernel releases its own dependents when it starts and calls griddepcontrol.wait only before
// its first write.  That is sound as long as nothing that may still be running wrote its inputs.  The
// only grids that release dependents early are this library's own, so the only writes that can still be
// in flight are the OUTPUTS of recent library calls of that kind.  Grids of this kind can pile up (each
// only needs its predecessor to have STARTED), so the record keeps every output buffer since the last
// call that waited first.  A call whose inputs overlap a recorded buffer, or whose outputs would not
// fit into the record, waits first; its grids then start only when everything before them is
// complete, which empties the record.
//
// Writes are ordered the same way.  A kernel that would write a buffer that a recorded call also writes
// has to know that call is over.  Calls of one context carry sequence numbers, and the context keeps a
// device word `done` = the largest sequence number whose call is known to be complete (written by a
// later call's kernel after ITS griddepcontrol.wait returned).  The launcher hands the kernel the number
// it needs (`need_seq`); the kernel writes at once when done >= need_seq and waits for the preceding
// grid otherwise.  Buffers written by anything that has no sequence number in that context make the
// kernel wait (need_seq = INT64_MAX).
#include <mutex>

#include "common.cuh"

namespace fedattn {

namespace {

constexpr int kRecord = 64;
struct Entry {
    MemRange r;
    const void *owner;      // whose sequence numbers `seq` counts in (a context's status area), or null
    int64_t seq;            // the owner's latest call that writes this buffer
};
struct OutputRecord {
    Entry e[kRecord];
    int n = 0;
};
OutputRecord g_outputs[64];        // per device
std::mutex g_outputs_mutex;

bool overlaps(const MemRange &a, const MemRange &b)
{
    const char *x = static_cast<const char *>(a.p), *y = static_cast<const char *>(b.p);
    return x && y && a.bytes && b.bytes && x < y + b.bytes && y < x + a.bytes;
}

}  // namespace

bool early_read_allowed(int device, const MemRange *in, int n_in, const MemRange *out, int n_out, const void *owner,
                        int64_t seq, int64_t *need_seq)
{
    std::lock_guard<std::mutex> lock(g_outputs_mutex);
    OutputRecord &rec = g_outputs[device & 63];
    bool wait_first = false;
    for (int i = 0; i < n_in && !wait_first; ++i)
        for (int j = 0; j < rec.n && !wait_first; ++j) wait_first = overlaps(in[i], rec.e[j].r);
    // Which recorded calls wrote into this call's outputs?  Calls of the same owner are named by their
    // sequence number (the kernel can tell on the device whether they are over); anything else cannot be
    // named and makes the call wait before its first write.
    int64_t need = 0;
    bool same[16];
    int n_new = 0;
    if (n_out > 16) wait_first = true;
    for (int o = 0; o < n_out && o < 16; ++o) {
        same[o] = false;
        if (!out[o].p || !out[o].bytes) continue;
        for (int j = 0; j < rec.n; ++j) {
            if (!overlaps(out[o], rec.e[j].r)) continue;
            if (owner && rec.e[j].owner == owner) need = need > rec.e[j].seq ? need : rec.e[j].seq;
            else need = INT64_MAX;
            if (rec.e[j].r.p == out[o].p && rec.e[j].r.bytes >= out[o].bytes && rec.e[j].owner == owner) {
                same[o] = true;
                rec.e[j].seq = seq;                               // the buffer's latest writer is this call
            }
        }
        n_new += !same[o];
    }
    if (rec.n + n_new > kRecord) wait_first = true;
    if (wait_first) { rec.n = 0; need = 0; }                      // this call waits first: nothing before it is left
    for (int o = 0; o < n_out && o < 16 && rec.n < kRecord; ++o)
        if (out[o].p && out[o].bytes && (wait_first || !same[o])) rec.e[rec.n++] = Entry{out[o], owner, seq};
    if (need_seq) *need_seq = need;
    return !wait_first;
}

}  // namespace fedattn
