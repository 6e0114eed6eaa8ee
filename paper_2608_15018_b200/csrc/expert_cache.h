// Residency of routed experts in a pool of device slots (expert-level offloading with hot experts
// kept resident: Sec. 5, "Edge memory constraints and expert-level offloading"): host-side
// bookkeeping only, no CUDA in here.
//
// Policy.  A layer has n_slots device slots.  Pinned experts (the offline profile's hot set) own
// slots 0 .. n_pinned-1 for good.  One access names the distinct experts a verification step
// activates; all of them must be resident at the same time, so none of them can be the victim of
// another.  Experts already resident are hits.  A missing expert takes the free slot of lowest
// index if there is one, else the unpinned slot that was used least recently and is not wanted by
// this access (ties: lowest slot index).  Misses are served in the order the experts are named.
#pragma once

#include <cstdint>
#include <vector>

namespace s2moe {

struct ExpertCache {
    int n_experts = 0, n_slots = 0, n_pinned = 0;
    std::vector<int32_t> slot_of;      // expert -> slot, -1 when not resident
    std::vector<int32_t> owner;        // slot -> expert, -1 when free
    std::vector<int64_t> last_use;     // slot -> number of the last access that used it (0: never)
    std::vector<int64_t> uses;         // expert -> accesses that named it
    int64_t clock = 0, hits = 0, misses = 0;

    // false when the arguments make no sense (range, duplicates, more pinned experts than slots)
    bool init(int E, int slots, const int32_t *pinned, int np)
    {
        if (E < 1 || slots < 1 || np < 0 || np > slots || np > E || (np > 0 && !pinned)) return false;
        n_experts = E; n_slots = slots; n_pinned = np;
        slot_of.assign((size_t)E, -1);
        owner.assign((size_t)slots, -1);
        last_use.assign((size_t)slots, 0);
        uses.assign((size_t)E, 0);
        clock = hits = misses = 0;
        for (int i = 0; i < np; ++i) {
            const int e = pinned[i];
            if (e < 0 || e >= E || slot_of[(size_t)e] >= 0) return false;
            slot_of[(size_t)e] = i;
            owner[(size_t)i] = e;
        }
        return true;
    }

    // One access: `experts` are n distinct expert ids.  Writes the slot of each and whether it had
    // to be fetched (1) or was resident (0).  Returns false, changing nothing, when the experts
    // cannot all be resident at once or an id is out of range or repeated.
    bool access(const int32_t *experts, int n, int32_t *slots_out, int32_t *missed_out)
    {
        if (n < 0 || n > n_slots) return false;
        std::vector<char> wanted((size_t)n_experts, 0);
        int need = 0;
        for (int i = 0; i < n; ++i) {
            const int e = experts[i];
            if (e < 0 || e >= n_experts || wanted[(size_t)e]) return false;
            wanted[(size_t)e] = 1;
            if (slot_of[(size_t)e] < 0) ++need;
        }
        // slots a missing expert may take: free ones and unpinned ones whose expert is not wanted
        int room = 0;
        for (int s = n_pinned; s < n_slots; ++s)
            if (owner[(size_t)s] < 0 || !wanted[(size_t)owner[(size_t)s]]) ++room;
        if (need > room) return false;
        ++clock;
        for (int i = 0; i < n; ++i) {
            const int e = experts[i];
            ++uses[(size_t)e];
            int s = slot_of[(size_t)e];
            if (s >= 0) {
                ++hits;
                missed_out[i] = 0;
            } else {
                ++misses;
                missed_out[i] = 1;
                s = -1;
                for (int c = n_pinned; c < n_slots && s < 0; ++c)
                    if (owner[(size_t)c] < 0) s = c;
                if (s < 0) {
                    for (int c = n_pinned; c < n_slots; ++c) {
                        if (wanted[(size_t)owner[(size_t)c]]) continue;
                        if (s < 0 || last_use[(size_t)c] < last_use[(size_t)s]) s = c;
                    }
                    slot_of[(size_t)owner[(size_t)s]] = -1;
                }
                owner[(size_t)s] = e;
                slot_of[(size_t)e] = s;
            }
            last_use[(size_t)s] = clock;
            slots_out[i] = s;
        }
        return true;
    }

    // Undo the residency of an expert whose weights did not arrive in its slot (a failed copy):
    // the slot is free again and the expert counts as not resident.  Pinned slots are left alone.
    void evict(int e)
    {
        if (e < 0 || e >= n_experts) return;
        const int s = slot_of[(size_t)e];
        if (s < n_pinned) return;            // not resident (-1) or pinned
        slot_of[(size_t)e] = -1;
        owner[(size_t)s] = -1;
        last_use[(size_t)s] = 0;
    }
};

}  // namespace s2moe
