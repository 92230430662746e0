"""Beam-pruning state machine, written out from the paper's description.  TEST INFRASTRUCTURE ONLY.

Sec. 4.2.2 ("New design in beam pruning"): the previous round's transcript tokens serve as a
reference for the current decoding session.

* search-based reference alignment -- decoding starts with beam size 1; the first top-1 token
  is searched through the reference list, the first match gives index i;
* selective token matching -- afterwards the top-1 token is compared with reference[i]: a match
  keeps the beam at 1 and advances i; a punctuation, timestamp or other special token is not
  compared at all (beam stays 1, i unchanged);
* fallback -- if the alignment search finds nothing, or a comparable token differs from
  reference[i], the beam returns to its full size.

Readings where the text leaves a choice (also listed in the design doc):
  R1  the alignment search uses the first top-1 token that is comparable (a leading timestamp or
      other special token is skipped like any other special token);
  R2  the aligned token counts as matched: after a hit at position i the next comparison is with
      reference[i + 1];
  R3  once the reference is exhausted a comparable token has nothing to match and triggers the
      fallback;
  R4  the fallback lasts until the end of the decoding session.
This module is independent of the library: plain Python, no shared code.
"""
from __future__ import annotations


class BeamPruner:
    def __init__(self, reference, special, full_beam=5):
        """reference: token ids of the previous round; special: set of ids that are never compared."""
        self.ref = list(reference)
        self.special = set(special)
        self.full = int(full_beam)
        self.i = None            # reference index once aligned
        self.fallen_back = False

    def step(self, top1: int) -> int:
        """Feed the top-1 token of a decoding round; returns the beam size for the NEXT round."""
        if self.fallen_back:
            return self.full
        if top1 in self.special:
            return 1
        if self.i is None:                                   # alignment search (R1)
            for pos, tok in enumerate(self.ref):
                if tok == top1:
                    self.i = pos + 1                          # R2
                    return 1
            self.fallen_back = True
            return self.full
        if self.i < len(self.ref) and self.ref[self.i] == top1:
            self.i += 1
            return 1
        self.fallen_back = True                               # mismatch, or reference exhausted (R3)
        return self.full


def run_session(reference, special, tokens, full_beam=5):
    """Beam size used in every round of a session (round 0 always runs with beam 1)."""
    p = BeamPruner(reference, special, full_beam)
    beams, nxt = [], 1
    for tok in tokens:
        beams.append(nxt)
        nxt = p.step(tok)
    return beams, p.i, p.fallen_back
