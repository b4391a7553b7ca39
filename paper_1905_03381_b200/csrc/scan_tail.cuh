// Shrink decision + order-preserving append shared by every scoring front end
// (Algorithm 1, Assistant.sample_batch, for a pool of candidates at once).
//
// Tiles of candidates are handed out in look-back order (a ticket counter; the bulk-copy kernel
// gives each CTA its block index as first tile and tickets after that); a tile's kept candidates
// are appended at the position given by a decoupled look-back over the tiles' counts.  A warp
// therefore only waits on tiles whose owners started before it or, for the block-index tiles, on
// CTAs of the same grid, which the launchers size to be resident together when the GPU is
// otherwise idle.  That is not a guarantee: if something else holds an SM (a scan of a second
// context on another stream, a foreign kernel's shared memory), a first tile's owner may not be
// running yet.  So every wait is bounded and gives up with a latched AA_ERR_SCAN_TIMEOUT instead
// of spinning for ever; the batch of such a call is invalid and the caller repeats it.
#pragma once

#include "aa_internal.cuh"

namespace aa {

__device__ __forceinline__ unsigned long long pack_state(unsigned int flag, int value) {
    return ((unsigned long long)flag << 32) | (unsigned int)value;
}

__device__ __forceinline__ unsigned int read_epoch(const ShrinkParams& p) {
    return *(volatile unsigned int*)&p.ctl->epoch;
}

// Row of candidate k, or -1 (latching AA_ERR_BAD_INDEX) when the candidate list points outside the store.
__device__ __forceinline__ long long candidate_row(const ShrinkParams& p, long long k) {
    if (!p.row_idx) return k;
    const long long r = p.row_idx[k];
    if ((unsigned long long)r >= (unsigned long long)p.n_stored) {
        latch(p.ctl, AA_ERR_BAD_INDEX);
        return -1;
    }
    return r;
}

// Keep/skip for candidate k with pre-activation s:  c < gamma + (1 - gamma) sigmoid(s),
// c drawn from Philox at counter (instance id, step).  Unreadable rows are skipped.
// In hard mode s is the instance's loss or gradient magnitude and the decision is s >= T.
__device__ __forceinline__ bool keep_decision(const ShrinkParams& p, long long k, float s) {
    long long r = k;
    if (p.row_idx) {
        r = p.row_idx[k];
        if ((unsigned long long)r >= (unsigned long long)p.n_stored) return false;
    }
    if (p.hard) return s >= p.hard_threshold;   // hard shrinking (Eq. "shrinking_grad"); NaN compares false
    const float prob = fmaf(1.0f - p.mix, sigmoid_f32(s), p.mix);
    const float c = philox_uniform(p, (uint64_t)(p.id_base + r));
    return c < prob;
}

// Decoupled look-back (warp-collective): publishes this tile's count and returns the number
// kept in all earlier tiles.
__device__ __forceinline__ int lookback_exclusive(const ShrinkParams& p, unsigned int tile, unsigned int epoch, int total) {
    const int lane = threadIdx.x & 31;
    const unsigned int flag_agg = epoch * 4u + 1u, flag_inc = epoch * 4u + 2u;
    unsigned long long* state = p.tile_state;
    if (tile == 0) {
        if (lane == 0) st_relaxed_u64(&state[0], pack_state(flag_inc, total));
        return 0;
    }
    if (lane == 0) st_relaxed_u64(&state[tile], pack_state(flag_agg, total));
    // Each poll reads the 32 predecessor states just before the window's end (lane l -> tile window_end - l) and the
    // window moves back by the groups that were complete.  Wider polls (256 states per round trip, to reach the
    // nearest finished prefix in one step when every SM runs in step) were measured: the extra loads of ~600 polling
    // warps cost the streaming kernels 7-9 % of their bandwidth and the scan-only kernels 10-20 % of their time.
    constexpr int kLookWide = 1;
    int excl = 0;          // committed sum of fully scanned groups (same in every lane)
    long long window_end = (long long)tile - 1;
    bool gave_up = false, found = false;
    unsigned int polls = 0;
    while (!found && !gave_up) {
        unsigned long long w[kLookWide];
#pragma unroll
        for (int j = 0; j < kLookWide; ++j) {
            const long long idx = window_end - j * 32 - lane;
            // tiles before tile 0 stand for "inclusive prefix 0"
            w[j] = idx >= 0 ? ld_relaxed_u64(&state[idx]) : pack_state(flag_inc, 0);
        }
        int lane_sum = 0, groups_done = 0;
        bool stalled = false;
#pragma unroll
        for (int j = 0; j < kLookWide; ++j) {
            if (!found && !stalled) {
                const unsigned int flag = (unsigned int)(w[j] >> 32);
                const int val = (int)(unsigned int)w[j];
                const unsigned int inc_m = __ballot_sync(0xFFFFFFFFu, flag == flag_inc);
                const unsigned int agg_m = __ballot_sync(0xFFFFFFFFu, flag == flag_agg);
                // only the tiles between this one and the nearest inclusive prefix have to be ready
                const int first = inc_m ? (__ffs(inc_m) - 1) : 31;
                const unsigned int need = inc_m ? ((1u << first) - 1u) : 0xFFFFFFFFu;
                if (((inc_m | agg_m) & need) == need) {
                    if (lane <= first) lane_sum += val;
                    ++groups_done;
                    found = inc_m != 0;
                } else {
                    stalled = true;
                }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) lane_sum += __shfl_xor_sync(0xFFFFFFFFu, lane_sum, o);
        excl += lane_sum;                       // groups before the stall are final: keep them
        window_end -= 32ll * groups_done;
        if (!found && stalled) {
            if (++polls > kSpinLimit) gave_up = true;
            else __nanosleep(polls < 64 ? 20 : 200);
        }
    }
    if (gave_up && lane == 0) latch(p.ctl, AA_ERR_SCAN_TIMEOUT);
    if (lane == 0) st_relaxed_u64(&state[tile], pack_state(flag_inc, excl + total));
    return excl;
}

// Last CTA out re-arms the ticket counter and starts a new flag generation, so the next
// scan on this context (a later launch on the same stream) needs no clearing pass.
__device__ __forceinline__ void scan_epilogue(const ShrinkParams& p, unsigned int epoch) {
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned int prev = atomicAdd(&p.ctl->done, 1u);
        if (prev == gridDim.x - 1) {
            p.ctl->ticket = 0;
            p.ctl->done = 0;
            unsigned int e = (epoch + 1u) & 0x3FFFFFFFu;
            p.ctl->epoch = e ? e : 1u;
        }
    }
}

// One warp finishes a whole tile of U*32 candidates whose pre-activations it holds in
// registers (lane l, unit u -> candidate k0 + u*32 + l): decisions, ballots, look-back, append.
template <int MAXU>
__device__ __forceinline__ void warp_shrink_compact(const ShrinkParams& p, unsigned int tile, unsigned int epoch,
                                                     int units, const float (&sv)[MAXU]) {
    const int lane = threadIdx.x & 31;
    const long long k0 = (long long)tile * p.tile_rows;
    unsigned int mask[MAXU];
    int total = 0;
#pragma unroll
    for (int u = 0; u < MAXU; ++u) {
        mask[u] = 0;
        if (u < units) {
            const long long k = k0 + u * 32 + lane;
            bool keep = false;
            if (u * 32 + lane < p.tile_rows && k < p.n_cand) {   // a tile may be shorter than a warp
                keep = keep_decision(p, k, sv[u]);
                if (p.out_score) p.out_score[k] = sv[u];
                if (p.out_mask) p.out_mask[k] = keep ? 1 : 0;
            }
            mask[u] = __ballot_sync(0xFFFFFFFFu, keep);
            total += __popc(mask[u]);
        }
    }
    const int base = lookback_exclusive(p, tile, epoch, total);
    if (lane == 0 && tile == p.n_tiles - 1) *p.out_count = base + total;
    int off = base;
#pragma unroll
    for (int u = 0; u < MAXU; ++u) {
        if (u < units) {
            const unsigned int m = mask[u];
            if ((m >> lane) & 1u) {
                const long long k = k0 + u * 32 + lane;
                const long long pos = (long long)off + __popc(m & ((1u << lane) - 1u));
                if (pos < p.capacity) p.out_idx[pos] = p.row_idx ? p.row_idx[k] : (int32_t)k;
                else latch(p.ctl, AA_ERR_CAPACITY);
            }
            off += __popc(m);
        }
    }
}

}  // namespace aa
