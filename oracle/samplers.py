"""ORACLE (test infrastructure): the LLaDA sampling strategies that Section 3.1 describes and that the paper's tables use
as the 1.00x baseline — random remasking, low-confidence remasking and semi-autoregressive remasking — in pure Python.

Each strategy is the transition S of Eq. 4: from the greedy estimate r_hat (and its confidences) of step k it decides
which [MASK] positions of y^(k) become tokens in y^(k-1); known tokens are always preserved.  Steps run k = N, N-1, .., 1.

  * Low-confidence remasking: y^(k-1) has n_un = floor(L * (1 - (k-1)/N)) unmasked positions, the n_un most confident
    ones, where an already decoded position has confidence 1.  Decoded positions therefore stay, and the step unmasks the
    n_un - (number already decoded) most confident masked positions (none if that is not positive).  "More confident" is
    "smaller canonical S_q" (see rowstats.c), ties to the smaller position; n_un is evaluated exactly in integers.
  * Random remasking: every masked position is unmasked with probability 1 - (k-1)/k = 1/k, independently.  The draws come
    from the counter-based generator Philox-4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2,
    3", SC'11) with key = the 64-bit seed and counter = (position, step index N - k, sequence index, 0); the position is
    unmasked iff  u * k < 2^32  for the first output word u — an integer comparison with probability ceil(2^32 / k) / 2^32.
  * Semi-autoregressive remasking: the response is cut into blocks of block_len positions (the last may be shorter), the N
    steps are divided evenly among the blocks (N must be a multiple of the number of blocks), and one of the two strategies
    above runs inside the current block — with the block's own length and step count in place of L and N — before the next
    block starts.  The predictor still sees the whole sequence; only the rows of the current block are read.

Readings (the paper describes the strategies in prose only): the steps of a block are N / n_blocks (how the reference LLaDA
sampler divides them is not in the paper); when every position is decoded before the steps run out (possible with random
remasking) the loop stops, since no later step could change the sequence.

Two statements again: whole-loop functions that follow the prose, and `vanilla_step`, a one-step state machine over the same
rule for a per-step entry point; the tests check one against the other.
"""
from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional, Sequence, Tuple

LOW_CONFIDENCE, RANDOM = 1, 2          # strategy ids (0 is SlowFast, see scheduler.py)
M32 = 0xFFFFFFFF


# ---- Philox-4x32-10 ------------------------------------------------------------------------------------------
PHILOX_M0, PHILOX_M1 = 0xD2511F53, 0xCD9E8D57        # round multipliers
PHILOX_W0, PHILOX_W1 = 0x9E3779B9, 0xBB67AE85        # key increments (golden ratio, sqrt 3 - 1)


def philox4x32_10(counter: Sequence[int], key: Sequence[int]) -> Tuple[int, int, int, int]:
    """Ten rounds of the Philox-4x32 bijection on a 128-bit counter under a 64-bit key."""
    c0, c1, c2, c3 = (int(c) & M32 for c in counter)
    k0, k1 = (int(k) & M32 for k in key)
    for _ in range(10):
        p0, p1 = PHILOX_M0 * c0, PHILOX_M1 * c2              # 64-bit products
        c0, c1, c2, c3 = ((p1 >> 32) ^ c1 ^ k0) & M32, p1 & M32, ((p0 >> 32) ^ c3 ^ k1) & M32, p0 & M32
        k0, k1 = (k0 + PHILOX_W0) & M32, (k1 + PHILOX_W1) & M32
    return c0, c1, c2, c3


def draw_accepts(u: int, k: int) -> bool:
    """Whether the 32-bit draw u unmasks at countdown k: u / 2^32 < 1 / k, i.e. exactly ceil(2^32 / k) of the 2^32 values do."""
    return u * k < (1 << 32)


def random_unmask(seed: int, seq: int, step_index: int, position: int, k: int) -> bool:
    """One Bernoulli(1/k) draw of random remasking: position `position` of sequence `seq` at step index N - k."""
    u = philox4x32_10((position, step_index, seq, 0), (seed & M32, (seed >> 32) & M32))[0]
    return draw_accepts(u, k)


# ---- the strategies, whole loops -------------------------------------------------------------------------------
Predict = Callable[[List[bool], List[int]], Tuple[Dict[int, int], Dict[int, int]]]
# predict(masked, rows) -> (a, sq): greedy token and canonical S_q for (at least) the positions in `rows`.


@dataclass
class VanillaRecord:
    step: int               # 0-based step index (N - k over the whole run)
    block: int
    k_block: int            # the block's own countdown (its N_b .. 1)
    positions: List[int]
    tokens: List[int]

    def key(self):
        return (self.step, self.block, self.k_block, tuple(self.positions), tuple(self.tokens))


def n_unmasked_target(L: int, N: int, k: int) -> int:
    """floor(L * (1 - (k-1)/N)), exactly."""
    return (L * (N - k + 1)) // N


def most_confident(cands: Sequence[int], sq: Dict[int, int], n: int) -> List[int]:
    return sorted(sorted(cands, key=lambda i: (int(sq[i]), i))[: max(n, 0)])


def _denoise_block(strategy: int, lo: int, hi: int, n_steps: int, masked: List[bool], y: List[Optional[int]], predict: Predict,
                   trace: List[VanillaRecord], block: int, seed: int, seq: int) -> None:
    """Applies one strategy to the positions [lo, hi) for n_steps steps (k = n_steps .. 1)."""
    Lb = hi - lo
    for k in range(n_steps, 0, -1):
        open_ = [i for i in range(lo, hi) if masked[i]]
        if not any(masked):
            return
        a, sq = predict(list(masked), open_) if open_ else ({}, {})
        if strategy == LOW_CONFIDENCE:
            have = Lb - len(open_)
            chosen = most_confident(open_, sq, n_unmasked_target(Lb, n_steps, k) - have)
        elif strategy == RANDOM:
            chosen = [i for i in open_ if random_unmask(seed, seq, len(trace), i, k)]
        else:
            raise ValueError("unknown strategy %r" % strategy)
        for i in chosen:
            masked[i] = False
            y[i] = int(a[i])
        trace.append(VanillaRecord(len(trace), block, k, chosen, [int(a[i]) for i in chosen]))


def semi_autoregressive(L: int, N: int, block_len: int, strategy: int, predict: Predict, seed: int = 0, seq: int = 0):
    """Section 3.1, semi-autoregressive remasking (block_len >= L gives the plain strategy).  Returns (tokens, trace)."""
    n_blocks = max(1, -(-L // block_len))
    if N % n_blocks:
        raise ValueError("N must be a multiple of the number of blocks")
    masked = [True] * L
    y: List[Optional[int]] = [None] * L
    trace: List[VanillaRecord] = []
    for j in range(n_blocks):
        _denoise_block(strategy, j * block_len, min(L, (j + 1) * block_len), N // n_blocks, masked, y, predict, trace, j, seed, seq)
    return y, trace


def low_confidence_remasking(L: int, N: int, predict: Predict):
    return semi_autoregressive(L, N, max(L, 1), LOW_CONFIDENCE, predict)


def random_remasking(L: int, N: int, predict: Predict, seed: int, seq: int = 0):
    return semi_autoregressive(L, N, max(L, 1), RANDOM, predict, seed, seq)


# ---- the same rule, one step at a time ---------------------------------------------------------------------------
@dataclass
class VanillaParams:
    strategy: int = LOW_CONFIDENCE
    max_steps: int = 0             # N; 0 means N = L
    block_len: int = 0             # 0 means one block (no semi-autoregressive split)
    seed: int = 0


@dataclass
class VanillaState:
    L: int
    N: int
    block_len: int
    steps_done: int = 0
    masked: List[bool] = field(default_factory=list)
    done: bool = False

    @staticmethod
    def fresh(L: int, p: VanillaParams) -> "VanillaState":
        N = p.max_steps if p.max_steps > 0 else L
        bl = p.block_len if 0 < p.block_len < L else max(L, 1)
        return VanillaState(L=L, N=N, block_len=bl, masked=[True] * L, done=(L == 0))

    @property
    def n_blocks(self):
        return max(1, -(-self.L // self.block_len))

    def block_span(self):
        """(block index, lo, hi, block-local k) of the NEXT step."""
        nb_steps = self.N // self.n_blocks
        j = self.steps_done // nb_steps
        return j, j * self.block_len, min(self.L, (j + 1) * self.block_len), nb_steps - self.steps_done % nb_steps


def vanilla_rows_needed(st: VanillaState) -> List[int]:
    if st.done:
        return []
    _, lo, hi, _ = st.block_span()
    return [i for i in range(lo, hi) if st.masked[i]]


def vanilla_step(st: VanillaState, a: Dict[int, int], sq: Dict[int, int], p: VanillaParams, seq: int = 0) -> Optional[VanillaRecord]:
    if st.done:
        return None
    j, lo, hi, k = st.block_span()
    open_ = [i for i in range(lo, hi) if st.masked[i]]
    if p.strategy == LOW_CONFIDENCE:
        nb_steps = st.N // st.n_blocks
        chosen = most_confident(open_, sq, n_unmasked_target(hi - lo, nb_steps, k) - ((hi - lo) - len(open_)))
    else:
        chosen = [i for i in open_ if random_unmask(p.seed, seq, st.steps_done, i, k)]
    for i in chosen:
        st.masked[i] = False
    rec = VanillaRecord(st.steps_done, j, k, chosen, [int(a[i]) for i in chosen])
    st.steps_done += 1
    if not any(st.masked) or st.steps_done >= st.N:
        st.done = True
    return rec
