// Online Correction Memory (Sec. 4.2): an open-addressed hash table in device memory
// mapping the ordered pair (draft token, target token) to a 32-bit count.
//
// Layout: n_slots (power of two) 16-byte slots {key:u64, count:u32, pad:u32}, linear
// probing from a 64-bit mix of the key.  An empty slot has key = ~0 (never a valid
// pair: both halves would be negative).  A look-up is one 16-byte load per probe.
//
// Capacity rule (this library's; the paper gives none): at most key_limit =
// n_slots / 2 distinct keys.  Present keys always count; new keys are admitted in
// the canonical (index) order of an update while there is room; an occurrence that
// finds no room is dropped and counted.  Because admission depends only on the set
// of keys and on the canonical order, the table's contents never depend on the hash
// function, on slot positions or on the order in which threads run.
#pragma once

#include "csd_common.cuh"

namespace csd {

struct __align__(16) OcmSlot {
    unsigned long long key;
    unsigned int count;
    unsigned int pad;
};

constexpr unsigned long long kEmptyKey = ~0ull;

struct OcmStatsDev {
    unsigned long long n_keys;        // distinct keys stored (live)
    unsigned long long n_keys_start;  // n_keys when the running update began (set between updates)
    unsigned long long n_dropped;
    unsigned long long steps;
    unsigned long long positions;
    unsigned long long matches;
    unsigned long long rescues;
    unsigned long long rejections;
    unsigned int flags;
    unsigned int ticket;              // arrival counter of multi-block update launches
    unsigned long long export_count;  // cursor of csd_ocm_export
    unsigned int debug_site;          // first failed index check (0 = none)
    unsigned int pad;
};

// Index checks.  A failed check sets a sticky flag, remembers which check it was and makes the
// caller skip the access; nothing traps.  CSD_CHECKED is for the one check that every build
// keeps; CSD_INDEX_OK compiles to `true` unless the library is built with -DCSD_DEBUG.
__device__ __noinline__ void index_check_failed(OcmStatsDev *stats, unsigned int site)
{
    atomicOr(&stats->flags, 0x10u);
    atomicCAS(&stats->debug_site, 0u, site);
}
#define CSD_CHECKED(cond, stats, site) ((cond) ? true : (csd::index_check_failed((stats), (site)), false))
#ifdef CSD_DEBUG
#define CSD_INDEX_OK(cond, stats, site) CSD_CHECKED(cond, stats, site)
#else
#define CSD_INDEX_OK(cond, stats, site) (true)
#endif

struct OcmView {
    OcmSlot *slots;
    unsigned long long mask;       // n_slots - 1
    unsigned long long key_limit;  // n_slots / 2
    unsigned int lambda;
    OcmStatsDev *stats;
    int shared;                    // 1: other streams may be updating the table while this launch runs
};

__device__ __forceinline__ unsigned long long make_key(int d, int t)
{
    return (static_cast<unsigned long long>(static_cast<unsigned int>(d)) << 32) |
           static_cast<unsigned long long>(static_cast<unsigned int>(t));
}

// 64-bit finaliser (xor-shift-multiply rounds); any well-mixing map works because
// the table's contents never depend on it.
__device__ __forceinline__ unsigned long long mix64(unsigned long long x)
{
    x ^= x >> 31;
    x *= 0x7fb5d329728ea185ull;
    x ^= x >> 27;
    x *= 0x81dadef4bc2dd44dull;
    x ^= x >> 33;
    return x;
}

__device__ __forceinline__ void load_slot(const OcmSlot *s, unsigned long long &key, unsigned int &count)
{
    const uint4 v = __ldcg(reinterpret_cast<const uint4 *>(s));
    key = (static_cast<unsigned long long>(v.y) << 32) | v.x;
    count = v.z;
}

// Count stored for `key`, 0 if absent.  *slot_out = slot index or -1; *empty_out = the empty
// slot that ended the probe of an absent key (where an insertion would begin), else -1.
__device__ __forceinline__ unsigned int ocm_lookup(const OcmView &tb, unsigned long long key, long long *slot_out = nullptr,
                                                   long long *empty_out = nullptr)
{
    if (empty_out) *empty_out = -1;
    unsigned long long slot = mix64(key) & tb.mask;
    for (unsigned long long probe = 0; probe <= tb.mask; ++probe) {
        unsigned long long k;
        unsigned int c;
        load_slot(tb.slots + slot, k, c);
        if (k == key) {
            if (slot_out) *slot_out = static_cast<long long>(slot);
            return c;
        }
        if (k == kEmptyKey) {
            if (slot_out) *slot_out = -1;
            if (empty_out) *empty_out = static_cast<long long>(slot);
            return 0;
        }
        slot = (slot + 1) & tb.mask;
    }
    atomicOr(&tb.stats->flags, 0x4u);
    if (slot_out) *slot_out = -1;
    return 0;
}

// count += w, saturating at 2^32 - 1.
__device__ __forceinline__ void ocm_add(const OcmView &tb, unsigned long long slot, unsigned int w)
{
    unsigned int *cnt = &tb.slots[slot].count;
    const unsigned int old = atomicAdd(cnt, w);
    if (old + w < old) {   // wrapped: pin to the maximum (every wrapping adder does the same)
        atomicExch(cnt, 0xffffffffu);
        atomicOr(&tb.stats->flags, 0x8u);
    }
}

// Insert-or-increment without a capacity check (the caller has established that there
// is room for every new key of the batch).
__device__ __forceinline__ void ocm_insert_or_add(const OcmView &tb, unsigned long long key, unsigned int w)
{
    unsigned long long slot = mix64(key) & tb.mask;
    for (unsigned long long probe = 0; probe <= tb.mask; ++probe) {
        unsigned long long *kp = &tb.slots[slot].key;
        unsigned long long k = *reinterpret_cast<volatile unsigned long long *>(kp);
        if (k == kEmptyKey) {
            k = atomicCAS(kp, kEmptyKey, key);
            if (k == kEmptyKey) {
                atomicAdd(&tb.stats->n_keys, 1ull);
                k = key;
            }
        }
        if (k == key) {
            ocm_add(tb, slot, w);
            return;
        }
        slot = (slot + 1) & tb.mask;
    }
    atomicOr(&tb.stats->flags, 0x4u);
}

// Slot of `key`, claiming an empty slot (count 0) if the key is absent.  A slot with
// count 0 reads as "absent" to every look-up, so a reservation is invisible until the
// count is raised.  The caller has established that there is room.  -1 only if the
// probe wrapped around (flagged).  `from` >= 0 is the empty slot at which a look-up of this
// key just ended: the probe resumes there (every slot before it holds another key, and
// keys never move or vanish) and tries to claim it without reading it again.
__device__ __forceinline__ long long ocm_reserve(const OcmView &tb, unsigned long long key, long long from = -1)
{
    unsigned long long slot = from >= 0 ? static_cast<unsigned long long>(from) : (mix64(key) & tb.mask);
    for (unsigned long long probe = 0; probe <= tb.mask; ++probe) {
        unsigned long long *kp = &tb.slots[slot].key;
        unsigned long long k = ~0ull;   // kEmptyKey: what the look-up saw at `from`
        if (!(from >= 0 && probe == 0)) k = *reinterpret_cast<volatile unsigned long long *>(kp);
        if (k == kEmptyKey) {
            k = atomicCAS(kp, kEmptyKey, key);
            if (k == kEmptyKey) {
                atomicAdd(&tb.stats->n_keys, 1ull);
                k = key;
            }
        }
        if (k == key) return static_cast<long long>(slot);
        slot = (slot + 1) & tb.mask;
    }
    atomicOr(&tb.stats->flags, 0x4u);
    return -1;
}

// ---- admission when several streams update one table at the same time ------------------------
// With a single writer the room for a batch's new keys is established before anyone inserts.  With
// concurrent writers every new key first takes one unit of the key budget from the live key count and
// gives it back if it turns out not to need it, so the table never holds more than key_limit keys
// whatever the interleaving; which keys get in near the limit then depends on arrival order.  Units
// that are held for the moment count against the room: while fewer keys of room remain than claims
// are in flight (at most B*K per step launch, 1024 per bulk update), a new key may be refused although
// room remains.  Far from the limit nothing is ever refused.
__device__ __forceinline__ bool ocm_take_key_budget(const OcmView &tb)
{
    const unsigned long long old = atomicAdd(&tb.stats->n_keys, 1ull);
    if (old < tb.key_limit) return true;
    atomicAdd(&tb.stats->n_keys, ~0ull);   // minus one
    return false;
}

// Slot of `key`, claiming an empty slot (count 0) if it is absent and the budget allows; -1 if the table
// is at its limit (or, flagged, if the probe wrapped around).  `from` as in ocm_reserve.
__device__ __forceinline__ long long ocm_reserve_shared(const OcmView &tb, unsigned long long key, long long from = -1)
{
    unsigned long long slot = from >= 0 ? static_cast<unsigned long long>(from) : (mix64(key) & tb.mask);
    bool budget = false;
    for (unsigned long long probe = 0; probe <= tb.mask; ++probe) {
        unsigned long long *kp = &tb.slots[slot].key;
        unsigned long long k = *reinterpret_cast<volatile unsigned long long *>(kp);
        if (k == kEmptyKey) {
            if (!budget) {
                if (!ocm_take_key_budget(tb)) return -1;
                budget = true;
            }
            k = atomicCAS(kp, kEmptyKey, key);
            if (k == kEmptyKey) return static_cast<long long>(slot);       // claimed: the budget unit is this key's
        }
        if (k == key) {
            if (budget) atomicAdd(&tb.stats->n_keys, ~0ull);               // somebody else brought the key in
            return static_cast<long long>(slot);
        }
        slot = (slot + 1) & tb.mask;
    }
    if (budget) atomicAdd(&tb.stats->n_keys, ~0ull);
    atomicOr(&tb.stats->flags, 0x4u);
    return -1;
}

__device__ __forceinline__ void ocm_insert_or_add_shared(const OcmView &tb, unsigned long long key, unsigned int w)
{
    const long long slot = ocm_reserve_shared(tb, key);
    if (slot >= 0)
        ocm_add(tb, static_cast<unsigned long long>(slot), w);
    else
        atomicAdd(&tb.stats->n_dropped, 1ull);
}

// Increment if present, else count a dropped occurrence (table full: nothing is admitted).
__device__ __forceinline__ void ocm_add_or_drop(const OcmView &tb, unsigned long long key, unsigned int w)
{
    long long slot;
    ocm_lookup(tb, key, &slot);
    if (slot >= 0)
        ocm_add(tb, static_cast<unsigned long long>(slot), w);
    else
        atomicAdd(&tb.stats->n_dropped, 1ull);
}

constexpr int kCanonChunk = 1024;   // entries handled at a time by the canonical-order path

struct CanonScratch {
    unsigned long long key[kCanonChunk];
    unsigned short first[kCanonChunk];
    unsigned char state[kCanonChunk];     // 0 done/skip, 1 pending first occurrence, 2 pending repeat
    unsigned char admit[kCanonChunk];
    unsigned long long avail;
};

__device__ __forceinline__ bool entry_key(const int *rd, const int *rt, long long j, unsigned long long &key)
{
    const int d = __ldcg(rd + j);
    const int t = __ldcg(rt + j);
    key = make_key(d, t);
    return d >= 0 && t >= 0;
}

// Canonical-order update of entries [j0, j0 + n) (n <= kCanonChunk) by the `nthreads`
// threads of one group (a whole block: `block_sync` true, or a single warp).  Used only
// while the table is close to its key limit, where the order of admission matters:
// new keys are ranked by their first occurrence and the first `avail` are admitted.
template <bool kBlock>
__device__ void ocm_update_canonical(const OcmView &tb, const int *rd, const int *rt, const unsigned int *w,
                                     long long j0, int n, CanonScratch &sc, int tid, int nthreads)
{
    auto sync = [&]() {
        if (kBlock) __syncthreads(); else __syncwarp();
    };
    if (tid == 0) {
        const unsigned long long nk = atomicAdd(&tb.stats->n_keys, 0ull);
        sc.avail = nk < tb.key_limit ? tb.key_limit - nk : 0ull;
    }
    // phase A: present keys count; absent ones become pending
    for (int j = tid; j < n; j += nthreads) {
        unsigned long long key;
        const bool valid = entry_key(rd, rt, j0 + j, key);
        sc.key[j] = key;
        unsigned char st = 0;
        if (valid) {
            long long slot;
            ocm_lookup(tb, key, &slot);
            if (slot >= 0)
                ocm_add(tb, static_cast<unsigned long long>(slot), w ? __ldcg(w + j0 + j) : 1u);
            else
                st = 1;
        }
        sc.state[j] = st;
        sc.admit[j] = 0;
    }
    sync();
    // phase B: mark repeats of a pending key and remember its first occurrence
    for (int j = tid; j < n; j += nthreads) {
        if (sc.state[j] == 0) continue;
        const unsigned long long key = sc.key[j];
        for (int i = 0; i < j; ++i) {
            if (sc.state[i] != 0 && sc.key[i] == key) {
                sc.first[j] = static_cast<unsigned short>(i);
                sc.state[j] = 2;
                break;
            }
        }
    }
    sync();
    // phase C: rank first occurrences in index order; the first `avail` are admitted
    for (int j = tid; j < n; j += nthreads) {
        if (sc.state[j] != 1) continue;
        unsigned long long rank = 0;
        for (int i = 0; i < j; ++i) rank += (sc.state[i] == 1);
        sc.admit[j] = rank < sc.avail;
    }
    sync();
    // phase D: admitted keys are inserted (repeats add to them); the rest are dropped
    for (int j = tid; j < n; j += nthreads) {
        const unsigned char st = sc.state[j];
        if (st == 0) continue;
        const int f = st == 1 ? j : sc.first[j];
        if (sc.admit[f])
            ocm_insert_or_add(tb, sc.key[j], w ? __ldcg(w + j0 + j) : 1u);
        else
            atomicAdd(&tb.stats->n_dropped, 1ull);
    }
    sync();
}

// UpdateMemory of Algorithm 1 for entries [0, n) by one group of threads that is the
// only writer of the table while it runs.  Three regimes, all giving the result of
// processing the entries one by one in index order:
//   room for everything   -> every thread inserts/increments independently
//   table full            -> increments only; absent keys are dropped
//   in between            -> canonical-order path, kCanonChunk entries at a time
template <bool kBlock>
__device__ void ocm_update_group(const OcmView &tb, const int *rd, const int *rt, const unsigned int *w,
                                 long long n, CanonScratch &sc, int tid, int nthreads)
{
    auto sync = [&]() {
        if (kBlock) __syncthreads(); else __syncwarp();
    };
    const unsigned long long nk = atomicAdd(&tb.stats->n_keys, 0ull);
    if (nk + static_cast<unsigned long long>(n) <= tb.key_limit) {
        for (long long j = tid; j < n; j += nthreads) {
            unsigned long long key;
            if (entry_key(rd, rt, j, key)) ocm_insert_or_add(tb, key, w ? __ldcg(w + j) : 1u);
        }
    } else if (nk >= tb.key_limit) {
        for (long long j = tid; j < n; j += nthreads) {
            unsigned long long key;
            if (entry_key(rd, rt, j, key)) ocm_add_or_drop(tb, key, w ? __ldcg(w + j) : 1u);
        }
    } else {
        for (long long j0 = 0; j0 < n; j0 += kCanonChunk) {
            const int cn = static_cast<int>(n - j0 < kCanonChunk ? n - j0 : kCanonChunk);
            sync();
            ocm_update_canonical<kBlock>(tb, rd, rt, w, j0, cn, sc, tid, nthreads);
        }
    }
    sync();
}

// ---- stand-alone kernels -------------------------------------------------------

__global__ void ocm_reset_kernel(OcmSlot *slots, unsigned long long n_slots, OcmStatsDev *stats)
{
    const unsigned long long stride = static_cast<unsigned long long>(gridDim.x) * blockDim.x;
    for (unsigned long long i = static_cast<unsigned long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < n_slots;
         i += stride) {
        uint4 v;
        v.x = 0xffffffffu;
        v.y = 0xffffffffu;
        v.z = 0u;
        v.w = 0u;
        *reinterpret_cast<uint4 *>(slots + i) = v;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        OcmStatsDev z = {};
        *stats = z;
    }
}

// csd_ocm_update / csd_ocm_import.  Every block reads the same n_keys_start (written
// when the previous update finished), so all blocks agree on the regime: with room
// for all n entries each block handles its slice; otherwise block 0 alone walks the
// whole batch in canonical order.  The last block to finish publishes n_keys_start.
__global__ void __launch_bounds__(1024) ocm_update_kernel(OcmView tb, const int *rd, const int *rt, const unsigned int *w,
                                                          long long n)
{
    __shared__ CanonScratch sc;
    __shared__ bool last;
    // Let a kernel launched programmatically behind this one begin (it waits in turn before it touches
    // the table), and, when launched programmatically behind the kernel that writes rd / rt, wait for
    // that one.  Both are no-ops for ordinary launches.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const unsigned long long nk0 = __ldcg(&tb.stats->n_keys_start);
    if (tb.shared) {
        // One block only: every thread that meets an absent key holds a unit of the key budget for the
        // duration of its claim, and a unit held is room that other writers cannot use meanwhile; a single
        // block bounds what one bulk update can hold at a time.
        if (blockIdx.x == 0) {
            for (long long j = threadIdx.x; j < n; j += blockDim.x) {
                unsigned long long key;
                if (entry_key(rd, rt, j, key)) ocm_insert_or_add_shared(tb, key, w ? __ldcg(w + j) : 1u);
            }
        }
    } else if (nk0 + static_cast<unsigned long long>(n) <= tb.key_limit) {
        const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
        for (long long j = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; j < n; j += stride) {
            unsigned long long key;
            if (entry_key(rd, rt, j, key)) ocm_insert_or_add(tb, key, w ? __ldcg(w + j) : 1u);
        }
    } else if (blockIdx.x == 0) {
        ocm_update_group<true>(tb, rd, rt, w, n, sc, threadIdx.x, blockDim.x);
    }
    if (tb.shared) return;     // other launches may be counting in as well; n_keys_start is not used while shared
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned int old = atomicAdd(&tb.stats->ticket, 1u);
        last = (old == gridDim.x - 1);
    }
    __syncthreads();
    if (last && threadIdx.x == 0) {
        __threadfence();
        const unsigned long long nk = atomicAdd(&tb.stats->n_keys, 0ull);
        tb.stats->n_keys_start = nk;
        tb.stats->ticket = 0u;
    }
}

// ---- ageing: every count halves (rounding down), pairs that reach zero are forgotten -----------
// Two launches.  The first moves the survivors (key, count / 2) to a side array and empties every
// slot; the second inserts them again, each at its own probe position in the emptied table (open
// addressing cannot delete in place: an emptied slot in the middle of a probe run would hide the keys
// behind it).  The table's contents never depend on slot positions, so the rebuilt table is the
// same table.  `cursor` (the statistics block's export cursor) counts the survivors.
__global__ void ocm_age_collect_kernel(OcmView tb, unsigned long long *keys, unsigned int *counts)
{
    const unsigned long long stride = static_cast<unsigned long long>(gridDim.x) * blockDim.x;
    for (unsigned long long i = static_cast<unsigned long long>(blockIdx.x) * blockDim.x + threadIdx.x; i <= tb.mask;
         i += stride) {
        unsigned long long k;
        unsigned int c;
        load_slot(tb.slots + i, k, c);
        if (k == kEmptyKey) continue;
        const unsigned int half = c >> 1;
        if (half) {
            const unsigned long long pos = atomicAdd(&tb.stats->export_count, 1ull);
            if (CSD_CHECKED(pos < tb.key_limit, tb.stats, 20u)) {     // at most key_limit pairs are ever stored
                keys[pos] = k;
                counts[pos] = half;
            }
        }
        uint4 v;
        v.x = 0xffffffffu; v.y = 0xffffffffu; v.z = 0u; v.w = 0u;
        __stcg(reinterpret_cast<uint4 *>(tb.slots + i), v);
    }
}

__global__ void ocm_age_reinsert_kernel(OcmView tb, const unsigned long long *keys, const unsigned int *counts)
{
    __shared__ bool last;
    unsigned long long n = __ldcg(&tb.stats->export_count);
    if (n > tb.key_limit) n = tb.key_limit;
    const unsigned long long stride = static_cast<unsigned long long>(gridDim.x) * blockDim.x;
    for (unsigned long long j = static_cast<unsigned long long>(blockIdx.x) * blockDim.x + threadIdx.x; j < n; j += stride) {
        const unsigned long long key = __ldcg(keys + j);
        unsigned long long slot = mix64(key) & tb.mask;
        bool placed = false;
        for (unsigned long long probe = 0; probe <= tb.mask; ++probe) {      // keys are distinct: claim the first empty slot
            if (atomicCAS(&tb.slots[slot].key, kEmptyKey, key) == kEmptyKey) {
                tb.slots[slot].count = __ldcg(counts + j);
                placed = true;
                break;
            }
            slot = (slot + 1) & tb.mask;
        }
        if (!placed) atomicOr(&tb.stats->flags, 0x4u);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        last = atomicAdd(&tb.stats->ticket, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (last && threadIdx.x == 0) {
        __threadfence();
        tb.stats->n_keys = n;
        tb.stats->n_keys_start = n;
        tb.stats->ticket = 0u;
    }
}

__global__ void ocm_export_kernel(OcmView tb, int *d, int *t, unsigned int *cnt, unsigned long long cap)
{
    const unsigned long long stride = static_cast<unsigned long long>(gridDim.x) * blockDim.x;
    for (unsigned long long i = static_cast<unsigned long long>(blockIdx.x) * blockDim.x + threadIdx.x; i <= tb.mask;
         i += stride) {
        unsigned long long k;
        unsigned int c;
        load_slot(tb.slots + i, k, c);
        if (k != kEmptyKey) {
            const unsigned long long pos = atomicAdd(&tb.stats->export_count, 1ull);
            if (pos < cap) {
                d[pos] = static_cast<int>(k >> 32);
                t[pos] = static_cast<int>(k & 0xffffffffull);
                cnt[pos] = c;
            }
        }
    }
}

}  // namespace csd
