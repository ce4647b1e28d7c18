// Greedy acceptance of one sequence's draft block (Section 3.2, Algorithm 1): the longest prefix on which the drafts
// equal the verifier's argmax tokens, then the verifier's token at the first mismatch.
#pragma once

#include <cstdint>

// d, t: the sequence's k draft / target ids; o: its k output ids.  kd = k, or k - 1 when the last row is the extra
// one (then a < k and t[a] is always emitted).  Returns the accepted length a; *n_emitted is the number of tokens
// in o (the rest of o is -1).  With eos_id >= 0 the output ends at the first eos token.
__device__ __forceinline__ int greedy_accept_row(const int32_t* __restrict__ d, const int32_t* __restrict__ t, int32_t* __restrict__ o,
                                                 int k, int kd, int32_t eos_id, int* n_emitted) {
    int a = 0;
    while (a < kd && d[a] == t[a]) ++a;
    int n = a < k ? a + 1 : a;
    for (int i = 0; i < k; ++i) o[i] = i < a ? d[i] : (i == a ? t[i] : -1);
    if (eos_id >= 0) {
        for (int i = 0; i < n; ++i)
            if (o[i] == eos_id) {
                for (int j = i + 1; j < n; ++j) o[j] = -1;
                n = i + 1;
                a = min(a, n);
                break;
            }
    }
    *n_emitted = n;
    return a;
}
