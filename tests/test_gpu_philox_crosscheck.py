"""The oracle's Philox4x32-10 against an independent implementation: the generator behind torch's CUDA random
numbers, which is the same published function keyed by the seed and counted by (offset, thread).  torch is asked
for raw 32-bit words (integers drawn from a range of exactly 2^32); every word it returns must be an output of
the oracle's function for the seed as key and some counter (call, 0, thread, 0).  This pins the round function,
the key schedule and the counter order with thousands of counters and keys the three published known answers do
not reach.  Tests only: nothing in the library uses torch's generator."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", [0, 1234, 2 ** 40 + 12345])
def test_oracle_philox_reproduces_the_words_of_torchs_cuda_generator(seed):
    from oracle import capi
    n = 2048
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    words = torch.randint(0, 2 ** 32, (n,), generator=gen, device="cuda", dtype=torch.int64).cpu().numpy()
    assert words.min() >= 0 and words.max() < 2 ** 32 and words.max() >= 2 ** 31      # full 32-bit words
    key = (seed & 0xFFFFFFFF, seed >> 32)
    candidates = set()
    for thread in range(8192):
        for call in range(4):
            candidates.update(capi.philox4x32_10((call, 0, thread, 0), key))
    found = sum(int(w) in candidates for w in words)
    # a word outside the set would be a different function; by chance a word is inside with probability 3e-5
    assert found == n, "%d of %d words of torch's generator are outputs of the oracle's Philox" % (found, n)
    # and a different key must not explain them
    other = set()
    for thread in range(512):
        other.update(capi.philox4x32_10((0, 0, thread, 0), (key[0] ^ 1, key[1])))
    assert sum(int(w) in other for w in words) <= 2
