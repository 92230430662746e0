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

Readings where the text leaves a choice:
  R1  the alignment search uses the first top-1 token that is comparable (a leading timestamp or
      other special token is skipped like any other special token);
  R2  the aligned token counts as matched: after a hit at position i the next comparison is with
      reference[i + 1];
  R3  once the reference is exhausted a comparable token has nothing to match and triggers the
      fallback;
  R4  the fallback lasts until the end of the decoding session;
  R5  punctuation, timestamp and special tokens are skipped on the reference side as well: the
      previous round's transcript carries them too, and a word must not be compared with a comma
      the model happened to emit last time.  The reference index rests right behind the last
      matched token; before a comparison it passes over special reference entries.
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
        j = self.i
        while j < len(self.ref) and self.ref[j] in self.special:     # R5
            j += 1
        if j < len(self.ref) and self.ref[j] == top1:
            self.i = j + 1
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
