"""Global beam selection, written out plainly (test infrastructure: only tests/, the smoke check and the CPU
baseline legs of bench.py may import this package; the CUDA path shares no code with it).

Section 2.1 of the paper: at each decoding step all active beams are expanded over the semantic-ID codebook and
the global top-k candidates are retained; several survivors may share a parent and other parents disappear, which
is what defines the parent map pi_t(b) that the ancestry index (Eq. 5) consumes.  The paper fixes nothing else,
so the reading taken here (and by the library) is:

  * a candidate (parent p, code c) scores  beam_score[p] + cand_logp[p, c], added in fp32 (the decision is taken
    in the precision the kernel uses);
  * the W_new best candidates are kept, best first;
  * equal scores are ordered by the smaller flat index p * C + c, so the result is unique;
  * a NaN score ranks below every number (and NaNs among themselves by flat index); -0.0 and +0.0 are equal.
"""
from __future__ import annotations

import numpy as np


def select_beams(beam_scores, cand_logp, W_new: int):
    """beam_scores [W_prev], cand_logp [W_prev, C] -> (parents [W_new] int32, codes [W_new] int32,
    scores [W_new] fp32), best first."""
    bs = np.asarray(beam_scores, dtype=np.float32)
    lp = np.asarray(cand_logp, dtype=np.float32)
    W_prev, C = lp.shape
    assert bs.shape == (W_prev,) and 1 <= W_new <= W_prev * C
    s = (bs[:, None] + lp).astype(np.float32).reshape(-1)
    nan = np.isnan(s)
    rank_key = np.where(nan, 0.0, s).astype(np.float64)
    # sort keys, most significant last: numbers before NaNs, then descending score, then ascending flat index
    order = np.lexsort((np.arange(s.size), -rank_key, nan.astype(np.int8)))[:W_new]
    return (order // C).astype(np.int32), (order % C).astype(np.int32), s[order]
