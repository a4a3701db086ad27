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
#include <mutex>

#include "common.cuh"

namespace fedattn {

namespace {

constexpr int kRecord = 64;
struct OutputRecord {
    MemRange r[kRecord];
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

bool early_read_allowed(int device, const MemRange *in, int n_in, const MemRange *out, int n_out)
{
    std::lock_guard<std::mutex> lock(g_outputs_mutex);
    OutputRecord &rec = g_outputs[device & 63];
    bool wait_first = false;
    for (int i = 0; i < n_in && !wait_first; ++i)
        for (int j = 0; j < rec.n && !wait_first; ++j) wait_first = overlaps(in[i], rec.r[j]);
    // outputs not yet covered by a recorded buffer
    bool is_new[16];
    int n_new = 0;
    if (n_out > 16) wait_first = true;
    for (int o = 0; o < n_out && o < 16; ++o) {
        is_new[o] = false;
        if (!out[o].p || !out[o].bytes) continue;
        bool known = false;
        for (int j = 0; j < rec.n && !known; ++j)
            known = rec.r[j].p == out[o].p && rec.r[j].bytes >= out[o].bytes;
        is_new[o] = !known;
        n_new += !known;
    }
    if (rec.n + n_new > kRecord) wait_first = true;
    if (wait_first) rec.n = 0;
    for (int o = 0; o < n_out && o < 16 && rec.n < kRecord; ++o)
        if (out[o].p && out[o].bytes && (wait_first || is_new[o])) rec.r[rec.n++] = out[o];
    return !wait_first;
}

}  // namespace fedattn
