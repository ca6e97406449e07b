"""Event-driven simulator of the ABS parameter-server loop (Algorithm 1).

Test infrastructure (see the package header).  One call of `run` plays rounds
t = 0, 1, ... of Algorithm 1 with U = 1 local step:

  (With `local_steps` = U > 1 a job is U local minibatch steps, Eq. 2: the worker
  starts from the model it holds, moves its own copy by -eta * (mean minibatch
  gradient) U times, each step on a fresh minibatch (in the bf16 configurations
  each step's gradient is evaluated at the bf16 rounding of that copy), and uploads the sum of its
  U mean gradients, i.e. (w^{.,0} - w^{.,U}) / eta, and the average of its U mean
  minibatch losses (Algorithm 1, last worker line); Eq. 3 is unchanged.)

  1. the server waits for the K^t fastest uploads (Sec. II-A; Algorithm 1,
     "waits for the uploads"): the K^t smallest pending completion events,
     ordered by (completion tick, worker id), ties to the lower id;
  2. each arriving worker k holds the model of the round it last downloaded,
     w^{t - tau_k}; its upload is the mean minibatch gradient of Eq. 2 at that
     model and its mean minibatch loss;
  3. global step, Eq. 3:  w^{t+1} = w^t - (eta / K^t) * sum_k g_k;
  4. the loss of the global model is taken to be the mean of the K^t uploaded
     losses (text below Eq. 5); K^{t+1} follows Eq. 5, floored, kept
     non-decreasing and at most N;
  5. threshold, Eq. 4, with the offset a chosen so that the initial threshold
     N/K^0 + a equals the staleness bound S:  theta = min(S, max(1, floor(N/K + a)));
  6. ages, Eq. 6 in the order Algorithm 1 performs it: arrivals get age 0; any
     other worker whose age after the increment exceeds theta is sent the new
     model and restarts its computation (its unfinished job is discarded);
  7. the communication counter grows by one per worker that talks to the
     server (Sec. V-B).

Comparison systems of the paper's evaluation (Sec. I, Sec. II-B, Sec. V) in the same loop:
  * AdaSync: K adapts as above but no worker is ever forced to restart (`restarts=False`), so
    the staleness of a consumed gradient is unbounded; the oracle keeps every model version
    some worker still holds.
  * Staleness-aware step size (SA): a stale gradient's step size is penalised linearly in its
    delay (`sa_penalty=True`): upload k enters Eq. 3 as g_k / max(1, tau_k).  SA-AdaSync is
    both switches together.

Symbols: N workers (W in the code), K, S, theta, B, eta as in the paper.
`version[n]` is the round index of the model worker n holds, so its age is
t - version[n].  Times are integer ticks (module `timing`).

Readings of passages the paper leaves open are spelled out next to the code
that implements them.
"""
import math
from fractions import Fraction

import numpy as np

from . import models, philox, timing

K_ADAPTIVE, K_FIXED = 0, 1
BOUND_ADAPTIVE, BOUND_FIXED, BOUND_OFFSET = 0, 1, 2


class Diverged(Exception):
    """A non-finite loss was uploaded; the run stops before that round's step."""


def shard_bounds(n, W, M):
    """Worker n's local dataset D_n: a contiguous slice of the M samples
    (disjoint slices whose union is the dataset, Sec. II-A)."""
    return (n * M) // W, ((n + 1) * M) // W


def minibatch_indices(seed, n, j, batch, W, M, step=0):
    """Sample indices of local step `step` of job j of worker n: independent
    uniform draws (with replacement) inside the worker's shard,
    index = lo + floor(r * len / 2**32)."""
    lo, hi = shard_bounds(n, W, M)
    words = philox.minibatch_words(seed, n, j, batch, step).astype(np.uint64)
    return lo + ((words * np.uint64(hi - lo)) >> np.uint64(32)).astype(np.int64)


def tree_sum(values):
    """Sum of binary32 numbers by adjacent pairs, level by level, after padding
    with zeros to a power of two; every addition is rounded to binary32.  The
    order and precision are part of the loss-estimate definition so that a
    parallel implementation gets the same bits."""
    v = [np.float32(x) for x in values]
    size = 1
    while size < len(v):
        size *= 2
    v += [np.float32(0.0)] * (size - len(v))
    while len(v) > 1:
        v = [np.float32(v[2 * i] + v[2 * i + 1]) for i in range(len(v) // 2)]
    return v[0]


def loss_estimate(upload_losses):
    """Estimate of f(w^t): mean of the uploaded binary32 losses, in binary32
    (the stored precision of every loss that decides an integer)."""
    k = len(upload_losses)
    return np.float32(tree_sum(upload_losses) / np.float32(k))


def next_k(k_now, k0, W, l0, lt):
    """Eq. 5 turned into an integer rule: the largest k in [1, N] with
    k <= K^0 sqrt(L0 / Lt), i.e. k^2 Lt <= K0^2 L0 (exact rational test on the
    stored binary32 losses), never below the current K (the analysis assumes
    K^0 <= K^t non-decreasing), never above N."""
    if not (math.isfinite(float(lt)) and math.isfinite(float(l0))):
        raise Diverged()
    if float(lt) <= 0.0:
        return W
    rhs = Fraction(k0 * k0) * Fraction(float(l0))
    k_raw = 0
    for k in range(1, W + 1):
        if Fraction(k * k) * Fraction(float(lt)) <= rhs:
            k_raw = k
    return min(W, max(k_now, k_raw))


def k_margin(k_now, k0, W, l0, lt):
    """Smallest relative distance |k^2 Lt - K0^2 L0| / (K0^2 L0) over the
    candidates k > k_now that could change the decision (diagnostic only)."""
    rhs = float(k0 * k0) * float(l0)
    best = math.inf
    for k in range(k_now + 1, W + 1):
        best = min(best, abs(float(k * k) * float(lt) - rhs) / rhs)
    return best


def theta_rule(W, k0, S, k):
    """Eq. 4 with a = S - N/K^0:  min(S, max(1, floor(N/K + a))), in exact
    rational arithmetic.  An age is an integer, so comparing it with the real
    threshold is the same as comparing it with the floor."""
    a = Fraction(S) - Fraction(W, k0)
    real_threshold = Fraction(W, k) + a
    return min(S, max(1, math.floor(real_threshold)))


def theta_offset_rule(W, S, k, a):
    """Eq. 4 as printed, with the constant a given: max{1, N/K + a}, floored
    (an integer age exceeds a real threshold iff it exceeds its floor; a is an
    integer here, as in the paper's experiments, Sec. V-B) and capped by the
    staleness bound S the model store is sized for."""
    return min(S, max(1, math.floor(Fraction(W, k) + a)))


class ABSOracle:
    """State of one simulated run.

    kind, dims     model kind (models.LSQ/SOFTMAX/MLP/CNN) and layer sizes (CNN: of its fully
                   connected part; `conv` = (H, W, C_in, k, C1, C2) describes the two convolution blocks)
    X, y           dataset; X either float array [M, in] or, with
                   `x_is_bf16_bits`, uint16 bfloat16 patterns
    w0             initial parameters (flat, layout of module `models`)
    batch, lr      B and eta
    W, K0, S       N workers, K^0, staleness bound
    dist, seed     time distribution and the Philox seed
    quant          round to bfloat16 at the storage points (bf16 configurations)
    k_mode         K_ADAPTIVE (Eq. 5) or K_FIXED
    bound_mode     BOUND_ADAPTIVE (Eq. 4 with a = S - N/K^0), BOUND_FIXED (theta = S
                   always) or BOUND_OFFSET (Eq. 4 with the integer `bound_offset` as a)
    local_steps    U of Eq. 2 (local minibatch steps per job)
    literal_eq6    test the pre-increment age against the threshold exactly as
                   Eq. 6 is printed (one round later than Algorithm 1's order)
    integer_only   play only the server's integer machinery (arrivals, Eq. 4-6,
                   ticks): no gradient is evaluated and the model stays at w^0;
                   every round must then be given its uploaded losses
    restarts       False: Eq. 6 never forces a restart (AdaSync, K-async SGD): ages grow until
                   the worker's own upload arrives; the threshold is still computed and recorded
    sa_penalty     staleness-aware step size: upload k is divided by max(1, tau_k) in Eq. 3
    """

    def __init__(self, kind, dims, X, y, w0, batch, lr, W, K0, S, dist, seed,
                 quant=False, k_mode=K_ADAPTIVE, bound_mode=BOUND_ADAPTIVE,
                 literal_eq6=False, x_is_bf16_bits=False, integer_only=False, bound_offset=0,
                 local_steps=1, restarts=True, sa_penalty=False, conv=None):
        if not (1 <= K0 <= W):
            raise ValueError("need 1 <= K0 <= W")
        if S < 0:
            raise ValueError("need S >= 0")
        self.kind, self.dims = kind, list(dims)
        self.X, self.y = X, y
        self.x_is_bf16_bits = x_is_bf16_bits
        self.M = X.shape[0]
        self.batch, self.lr = int(batch), float(lr)
        self.W, self.K0, self.S = int(W), int(K0), int(S)
        self.dist, self.seed = dist, int(seed)
        self.quant = bool(quant)
        self.k_mode, self.bound_mode = k_mode, bound_mode
        self.bound_offset = int(bound_offset)
        self.local_steps = int(local_steps)
        if self.local_steps < 1:
            raise ValueError("need U >= 1")
        if bound_mode == BOUND_OFFSET and theta_offset_rule(self.W, 10 ** 9, self.K0, self.bound_offset) > self.S:
            raise ValueError("staleness bound below the initial threshold N/K0 + a")
        self.literal_eq6 = literal_eq6
        self.integer_only = integer_only
        self.restarts = bool(restarts)
        self.sa_penalty = bool(sa_penalty)
        self.w = np.array(w0, dtype=np.float64)
        self.conv = None if conv is None else tuple(int(v) for v in conv)
        if kind == models.CNN:
            assert self.w.shape[0] == models.cnn_n_params(self.conv, dims)
        else:
            assert self.w.shape[0] == models.n_params(kind, dims)
        # the oracle may keep every past model; the bound is what lets a real
        # implementation keep only S + 1 of them
        self.versions = {0: self._stored(self.w)}
        self.t = 0
        self.K = self.K0
        self.L0 = None
        self.version = [0] * self.W
        self.job = [0] * self.W
        self.c = [timing.duration_ticks(dist, self.seed, n, 0) for n in range(self.W)]
        self.comm = self.W          # the initial broadcast reaches every worker
        self.min_margin = math.inf
        self.trace = []

    # -- helpers -----------------------------------------------------------
    def _stored(self, w):
        """The copy of the global model that workers download."""
        return models.round_bf16(w) if self.quant else w.copy()

    def _rows(self, idx):
        rows = self.X[idx]
        if self.x_is_bf16_bits:
            rows = (rows.astype(np.uint32) << np.uint32(16)).view(np.float32)
        return rows.astype(np.float64)

    def upload(self, n):
        """Upload of worker n's current job (Eq. 2): the average of the U mean
        minibatch losses and the sum of the U mean minibatch gradients along the
        worker's local trajectory, which starts at the model version it holds."""
        held = self.versions[self.version[n]]        # the stored copy the worker downloaded
        w_local = np.array(held, dtype=np.float64)
        loss_sum, grad_sum = 0.0, np.zeros_like(w_local)
        for u in range(self.local_steps):
            idx = minibatch_indices(self.seed, n, self.job[n], self.batch, self.W, self.M, step=u)
            Xb = self._rows(idx)
            yb = self.y[idx]
            if self.kind == models.LSQ:
                yb = yb.astype(np.float64)
            # bf16 configurations compute every step with the 16-bit rounding of the local copy
            # (the copy itself keeps full precision); at step 0 that is the downloaded model, which
            # is stored rounded already (rounding it again would change nothing)
            w_eval = held if u == 0 else self._stored(w_local)
            loss, grad = models.loss_grad(self.kind, self.dims, w_eval, Xb, yb, quant=self.quant, conv=self.conv)
            loss_sum += loss
            grad_sum += grad
            if u + 1 < self.local_steps:
                w_local = w_local - self.lr * grad                       # Eq. 2
        return loss_sum / self.local_steps, grad_sum

    def _start_job(self, n, now):
        """Worker n receives w^{t+1} at tick `now` and starts its next job."""
        self.version[n] = self.t + 1
        self.job[n] += 1
        self.c[n] = now + timing.duration_ticks(self.dist, self.seed, n, self.job[n])
        if self.c[n] >= timing.MAX_TICKS:
            raise OverflowError("simulated time out of tick range")

    # -- one round ---------------------------------------------------------
    def round(self, forced_losses=None):
        """Play round t.  `forced_losses` (binary32, arrival order) replaces the
        oracle's own uploaded losses in the K rule only; used to check the
        integer machinery against a run whose floating-point losses differ in
        the last bits."""
        t, K = self.t, self.K
        # every worker has exactly one job in flight; its completion tick is c[n]
        arrivals = sorted(range(self.W), key=lambda n: (self.c[n], n))[:K]
        T_end = self.c[arrivals[-1]]
        taus = [t - self.version[n] for n in arrivals]

        own_losses, grad_sum = [], np.zeros_like(self.w)
        if self.integer_only:
            assert forced_losses is not None and len(forced_losses) == K
            own_losses = [np.float32(x) for x in forced_losses]
        else:
            for n, tau in zip(arrivals, taus):
                loss, grad = self.upload(n)
                own_losses.append(np.float32(loss))
                if self.sa_penalty:
                    grad = grad / max(1, tau)          # step size penalised linearly in the delay
                grad_sum += grad
        losses = own_losses if forced_losses is None else \
            [np.float32(x) for x in forced_losses]
        if not all(math.isfinite(float(x)) for x in losses):
            raise Diverged()

        if not self.integer_only:
            self.w = self.w - (self.lr / K) * grad_sum                  # Eq. 3
            self.versions[t + 1] = self._stored(self.w)

        Lt = loss_estimate(losses)
        if t == 0:
            self.L0 = Lt             # f(w^0): every round-0 upload was computed at w^0
        if self.k_mode == K_ADAPTIVE:
            self.min_margin = min(self.min_margin, k_margin(K, self.K0, self.W, self.L0, Lt))
            K_next = next_k(K, self.K0, self.W, self.L0, Lt)            # Eq. 5
        else:
            K_next = K
        if self.bound_mode == BOUND_ADAPTIVE:
            theta = theta_rule(self.W, self.K0, self.S, K_next)         # Eq. 4
        elif self.bound_mode == BOUND_OFFSET:
            theta = theta_offset_rule(self.W, self.S, K_next, self.bound_offset)
        else:
            theta = self.S

        selected = set(arrivals)
        restarted = []
        for n in range(self.W):                                         # Eq. 6
            if n in selected:
                continue
            age_now = t - self.version[n]
            over = (age_now > theta) if self.literal_eq6 else (age_now + 1 > theta)
            if over and self.restarts:
                restarted.append(n)
        for n in arrivals + restarted:
            self._start_job(n, T_end)
        # drop model copies that no worker holds any more (memory only)
        for v in [v for v in self.versions if v not in set(self.version) and not self.integer_only]:
            del self.versions[v]
        self.comm += K + len(restarted)

        row = dict(t=t, K=K, sel=list(arrivals), tau=taus, restart=restarted,
                   T_end=T_end, theta=theta, loss_mean=float(Lt),
                   sel_loss=[float(x) for x in own_losses], comm=self.comm,
                   K_next=K_next)
        self.trace.append(row)
        self.K = K_next
        self.t = t + 1
        return row

    def run(self, n_rounds, forced_losses=None):
        """Play n_rounds rounds; `forced_losses[i]` (optional) feeds round i of
        this call.  Returns the rows appended."""
        first = len(self.trace)
        for i in range(n_rounds):
            self.round(None if forced_losses is None else forced_losses[i])
        return self.trace[first:]
