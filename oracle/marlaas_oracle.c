/* CPU oracle for the multi-tenant LoRA linear layer -- TEST INFRASTRUCTURE ONLY.
 *
 * Plain C loops written from the layer's definition (see marlaas_oracle_impl.inc for the
 * equations).  It shares no code with the CUDA library; only tests, the smoke check and the
 * benchmark's cpu_baseline / reference legs may call it.  The product path never does.
 *
 * Every function here is pinned by tests/test_oracle_pins.py (zero-B, merged weight, token
 * permutation, rank-1 closed form, finite differences, adjoint identities, routing probe,
 * scale doubling, rank padding, brute-force index build).
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define REAL float
#define SUFFIX _f32
#include "marlaas_oracle_impl.inc"
#undef REAL
#undef SUFFIX

#define REAL double
#define SUFFIX _f64
#include "marlaas_oracle_impl.inc"
#undef REAL
#undef SUFFIX

int marlaas_oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Index build from the token-to-adapter segment table.
 *   seg_offsets[S+1] (first 0, non-decreasing, last T), seg_slot[S] in [-1, cap)
 *   tok_slot[i]    = slot of the segment that contains token i
 *   slot_count[t]  = tokens of slot t for t in [0,cap); slot_count[cap] counts slot -1
 *   slot_offset    = exclusive prefix sum of slot_count in the order 0..cap-1, then -1 (cap+2 entries,
 *                    the last one equals T)
 *   perm           = token indices stably sorted by that key (ascending token index within a slot)
 * Returns 0, or -1 if the table is malformed. */
int marlaas_oracle_build_index(int T, int S, const int32_t* seg_offsets, const int32_t* seg_slot, int cap,
                               int32_t* tok_slot, int32_t* slot_count, int32_t* slot_offset, int32_t* perm) {
    if (T < 0 || S < 0 || seg_offsets[0] != 0 || seg_offsets[S] != T) return -1;
    for (int s = 0; s < S; ++s) {
        if (seg_offsets[s + 1] < seg_offsets[s]) return -1;
        if (seg_slot[s] < -1 || seg_slot[s] >= cap) return -1;
    }
    for (int s = 0; s < S; ++s)
        for (int i = seg_offsets[s]; i < seg_offsets[s + 1]; ++i) tok_slot[i] = seg_slot[s];
    for (int t = 0; t <= cap; ++t) slot_count[t] = 0;
    for (int i = 0; i < T; ++i) slot_count[tok_slot[i] < 0 ? cap : tok_slot[i]] += 1;
    slot_offset[0] = 0;
    for (int t = 0; t <= cap; ++t) slot_offset[t + 1] = slot_offset[t] + slot_count[t];
    int32_t* cursor = (int32_t*)malloc(sizeof(int32_t) * (size_t)(cap + 1));
    memcpy(cursor, slot_offset, sizeof(int32_t) * (size_t)(cap + 1));
    for (int i = 0; i < T; ++i) {
        const int key = tok_slot[i] < 0 ? cap : tok_slot[i];
        perm[cursor[key]++] = i;
    }
    free(cursor);
    return 0;
}
