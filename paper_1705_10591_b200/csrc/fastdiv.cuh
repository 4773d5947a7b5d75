// Division by a divisor that is fixed per launch, without a division instruction.
#pragma once

#include <stdint.h>

namespace conv2d_b200 {

// Division of a non-negative int below 2^31 by a divisor fixed per launch, as a multiply-high, an add and a
// shift (round-up method for invariant divisors): a plain 32-bit division is a ~35-instruction dependent chain,
// and index decoding sits on the critical path of the threads that feed and drain the tensor cores.
struct FastDiv {
    uint32_t mul, shift;
    int d;
    FastDiv() : mul(0), shift(0), d(1) {}
    explicit FastDiv(int divisor) : d(divisor)
    {
        uint32_t l = 0;
        while ((1ull << l) < (unsigned long long)divisor) ++l;
        shift = l;
        mul = (uint32_t)((((1ull << l) - (unsigned long long)divisor) << 32) / (unsigned long long)divisor + 1ull);
    }
    __device__ __forceinline__ int div(int n) const { return (int)((__umulhi((uint32_t)n, mul) + (uint32_t)n) >> shift); }
    __device__ __forceinline__ int divmod(int n, int& rem) const { const int q = div(n); rem = n - q * d; return q; }
};

}  // namespace conv2d_b200
