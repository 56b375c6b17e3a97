// Phrase-key formation and bucket hashing, shared by the host-side index build
// and the device kernels of the library (never by the CPU oracle).
//
// A phrase key is derived from the token ids of an n-gram (paper Sec. 2.2 names token
// n-grams as a source of keys).  The memory must be exact -- one
// logical entry per phrase, no shared slots (Sec. 3.1) -- so a key identifies a
// token tuple, not a hash class:
//   * an order n with n * bits_per_token <= 61 is PACKED: the ids are laid side
//     by side under a 3-bit order tag.  Distinct tuples give distinct keys.
//   * a longer order is HASHED into 61 bits under the same tag.  The build
//     refuses two tuples with one key and a lookup confirms a key match against
//     the stored tuple, so the mapping stays exact.
// The tag is 1..4, hence a key is never 0 and 0 marks an empty index slot.
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define TFE_HD __host__ __device__ __forceinline__
#else
#define TFE_HD inline
#endif

#define TFE_SLOTS_PER_BUCKET 4
#define TFE_TAG_SHIFT 61

TFE_HD uint64_t tfe_mix64(uint64_t z)
{
    z ^= z >> 33; z *= 0xFF51AFD7ED558CCDull;
    z ^= z >> 33; z *= 0xC4CEB9FE1A85EC53ull;
    z ^= z >> 33;
    return z;
}

TFE_HD int tfe_token_bits(int32_t vocab)
{
    int b = 1;
    while (b < 31 && (1ll << b) < (long long)vocab) ++b;
    return b;
}

TFE_HD bool tfe_order_is_packed(int n, int tok_bits) { return n * tok_bits <= TFE_TAG_SHIFT; }

// tk[j] = token at distance j before the query position (tk[0] is the last token
// of the n-gram); all of tk[0..n) must be valid ids.
TFE_HD uint64_t tfe_make_key(int n, const int32_t tk[4], int tok_bits)
{
    uint64_t acc;
    if (tfe_order_is_packed(n, tok_bits)) {
        acc = 0;
#pragma unroll
        for (int j = 3; j >= 0; --j)
            if (j < n) acc = (acc << tok_bits) | (uint64_t)(uint32_t)tk[j];
    } else {
        acc = 0x2545F4914F6CDD1Dull;
#pragma unroll
        for (int j = 3; j >= 0; --j)
            if (j < n) acc = tfe_mix64(acc ^ ((uint64_t)(uint32_t)tk[j] + 0x9E3779B97F4A7C15ull));
        acc >>= 64 - TFE_TAG_SHIFT;
    }
    return ((uint64_t)n << TFE_TAG_SHIFT) | acc;
}

// The two buckets a key may live in (bucketed cuckoo hashing, 4 slots of 16 bytes per bucket).
// Each is a multiply-high range reduction of a mixed key, so any bucket count (not only powers
// of two) is covered evenly; the second is forced to differ from the first.
TFE_HD uint64_t tfe_mulhi64(uint64_t a, uint64_t b)
{
#if defined(__CUDA_ARCH__)
    return __umul64hi(a, b);
#else
    return (uint64_t)(((unsigned __int128)a * b) >> 64);
#endif
}

TFE_HD uint64_t tfe_home_bucket_of(uint64_t key, uint64_t n_buckets)
{
    return tfe_mulhi64(tfe_mix64(key), n_buckets);
}

TFE_HD uint64_t tfe_second_bucket_of(uint64_t key, uint64_t first, uint64_t n_buckets)
{
    uint64_t b = tfe_mulhi64(tfe_mix64(key ^ 0xD6E8FEB86659FD93ull), n_buckets);
    if (b == first) b = b + 1 == n_buckets ? 0 : b + 1;
    return b;
}
