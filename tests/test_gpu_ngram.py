"""The prompt-lookup drafter on the GPU against the oracle (Section 4.1), bit for bit."""
import numpy as np
import pytest
import torch

from oracle import quasar_oracle as qo
from paper_2603_01399_b200 import binding

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("alphabet,S,gamma,k", [(3, 64, 5, (1, 3)), (50, 700, 7, (2, 4)), (1000, 4096, 9, (1, 4)), (2, 33, 3, (3, 5))])
def test_ngram_draft_matches_the_oracle(alphabet, S, gamma, k):
    rng = np.random.default_rng(alphabet + S)
    B = 32
    hist = rng.integers(0, alphabet, (B, S)).astype(np.int32)
    # half of the sequences repeat a phrase, as code or a quoted prompt does
    for b in range(0, B, 2):
        period = int(rng.integers(3, 40))
        hist[b] = np.resize(hist[b, :period], S)
    lens = rng.integers(0, S + 1, B).astype(np.int32)
    lens[0], lens[1], lens[2] = S, 1, 0
    draft, dlen = binding.quasar_ngram_draft(torch.from_numpy(hist).cuda(), torch.from_numpy(lens).cuda(), gamma, k[0], k[1])
    draft, dlen = draft.cpu().numpy(), dlen.cpu().numpy()
    for b in range(B):
        want = qo.ngram_draft(hist[b, :lens[b]], gamma, k[0], k[1])
        assert dlen[b] == len(want), (b, dlen[b], want)
        assert list(draft[b, :len(want)]) == want and np.all(draft[b, len(want):] == -1)
    assert dlen[::2].mean() > dlen[1::2].mean() or alphabet <= 3
