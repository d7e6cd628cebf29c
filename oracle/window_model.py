"""Sliding-window memory scheduler: sizes and timeline.  TEST INFRASTRUCTURE ONLY.

Host-only statements of what Sec. 3.3 and Appendices A.3-A.5 define, used to
pin the GPU library's window accounting (block byte sizes, slot counts, order
of loads, stalls).  Imports nothing from the product.

* ``block_params``    - Table 5: parameters per block for a device owning a
                        fraction p of the heads / FFN columns.
* ``worker_peak``     - Prop. 5, M_worker without the empirical factor gamma.
* ``master_peak``     - Prop. 5, M_master without gamma.
* ``timeline``        - the time-slot model of the proof of Prop. 3: one loader
                        that loads blocks one after another in execution order,
                        a window of w blocks (the executing one included), a
                        block released after its compute and its allreduce.
* ``loose_condition`` / ``tight_condition`` - Prop. 3 / Prop. 4 as printed.
"""
from __future__ import annotations


def block_params(kind: str, h: int, v: int, a: int, b: int, s: int, p: float) -> float:
    """Table 5.  kind in {"pre", "attn", "ffn", "post"}."""
    if kind == "pre":
        return h * v
    if kind == "attn":
        return 2 * (a + b) * h * h * p / a + h
    if kind == "ffn":
        return 3 * h * s * p + h
    if kind == "post":
        return h * v + h
    raise ValueError(kind)


def worker_peak(w: int, h: int, a: int, b: int, s: int, p: float) -> float:
    """Prop. 5: floor(w/2) attention blocks + floor((w+1)/2) FFN blocks (in parameters)."""
    attn = 2 * (1 + b / a) * h * h * p + h
    ffn = 3 * h * s * p + h
    return (w // 2) * attn + ((w + 1) // 2) * ffn


def master_peak(w: int, h: int, v: int, a: int, b: int, s: int, p: float) -> float:
    """Prop. 5, master: pre/postprocess blocks take window places too."""
    if w == 1:
        return h * v + h
    if w == 2:
        return 2 * h * v + h
    attn = 2 * (1 + b / a) * h * h * p + h
    ffn = 3 * h * s * p + h
    return 2 * h * v + h + ((w - 2) // 2) * attn + ((w - 1) // 2) * ffn


def timeline(t_attn, t_ffn, t_ar, tau_attn, tau_ffn, n_blocks: int, w: int):
    """Discrete-event model of Appendix A.3's time slots.

    Blocks alternate attention, FFN, attention, ... (block 0 is attention).
    The loader starts at time 0, loads block k for tau_k, one block at a time,
    in order, and may not begin block k before block k-w has been released
    (the window holds at most w blocks, the executing one included).
    Block k computes for t_k once it is loaded and block k-1 (with its
    allreduce) is done; it is released when its allreduce ends.

    Returns (stall, slack, end): per block, how long compute waited for the
    weights, how long the weights were ready ahead of need (the proof's t'
    when positive), and the total time.
    """
    load_done = [0.0] * n_blocks
    released = [0.0] * n_blocks
    stall = [0.0] * n_blocks
    slack = [0.0] * n_blocks
    loader_free = 0.0
    prev_done = 0.0
    for k in range(n_blocks):
        is_attn = (k % 2 == 0)
        tau = tau_attn if is_attn else tau_ffn
        t = t_attn if is_attn else t_ffn
        start_load = loader_free if k < w else max(loader_free, released[k - w])
        load_done[k] = start_load + tau
        loader_free = load_done[k]
        ready = prev_done
        stall[k] = max(0.0, load_done[k] - ready)
        slack[k] = max(0.0, ready - load_done[k])
        begin = max(ready, load_done[k])
        released[k] = begin + t + t_ar
        prev_done = released[k]
    return stall, slack, prev_done


def loose_condition(t_attn, t_ffn, t_ar, tau_attn, tau_ffn, L: int) -> bool:
    """Prop. 3."""
    if t_attn + t_ffn + 2 * t_ar < tau_ffn + tau_attn:
        return False
    first = all(l * t_attn + (l - 1) * t_ffn + (2 * l - 1) * t_ar >= l * tau_ffn + (l - 1) * tau_attn
                for l in range(1, L + 1))
    second = all((l - 1) * t_attn + l * t_ffn + (2 * l - 1) * t_ar >= (l - 1) * tau_ffn + l * tau_attn
                 for l in range(1, L + 1))
    return first or second


def tight_condition(t_attn, t_ffn, t_ar, tau_attn, tau_ffn) -> bool:
    """Prop. 4."""
    return t_attn + t_ar >= tau_ffn and t_ffn + t_ar >= tau_attn


def retained_ffn_layers(L: int, T: int):
    """Appendix A.6's indicator: with one FFN block kept in every T, the kept ones are those of
    layers l = 1 + kT (1-based), i.e. 0, T, 2T, ... (0-based).  T = 0: none."""
    return set() if T <= 0 else set(range(0, L, T))


def timeline_retained(t_attn, t_ffn, t_ar, tau_attn, tau_ffn, n_blocks: int, w: int, T: int, L: int):
    """The time-slot model with block retention (Prop. 6 / Appendix A.6).

    As ``timeline`` (blocks alternate attention, FFN; execution wraps around after 2L blocks), except
    that the FFN blocks of the retained layers are always in memory: the loader skips them and they
    never wait.  The window's w places are split as Prop. 5 counts them, floor(w/2) attention and
    ceil(w/2) FFN blocks (w = 1: a single shared place), so a streamed block may start loading only
    after the streamed block of its kind that many places earlier has been released.
    """
    keep = retained_ffn_layers(L, T)
    n_slots = {0: w // 2, 1: (w + 1) // 2} if w > 1 else None
    stall = [0.0] * n_blocks
    slack = [0.0] * n_blocks
    released_of_kind = {0: [], 1: [], 2: []}      # release times of streamed blocks, per kind (2: shared, w = 1)
    loader_free = 0.0
    prev_done = 0.0
    for k in range(n_blocks):
        kind = k % 2
        layer = (k // 2) % L
        t = t_ffn if kind else t_attn
        if kind == 1 and layer in keep:
            prev_done += t + t_ar
            continue
        tau = tau_ffn if kind else tau_attn
        hist = released_of_kind[kind if n_slots else 2]
        places = n_slots[kind] if n_slots else 1
        start_load = loader_free if len(hist) < places else max(loader_free, hist[len(hist) - places])
        load_done = start_load + tau
        loader_free = load_done
        stall[k] = max(0.0, load_done - prev_done)
        slack[k] = max(0.0, prev_done - load_done)
        prev_done = max(prev_done, load_done) + t + t_ar
        hist.append(prev_done)
    return stall, slack, prev_done


def retention_condition(t_attn, t_ffn, t_ar, tau_attn, tau_ffn, L: int, T: int) -> bool:
    """Prop. 6 as printed: both families of inequalities for l = 1..L."""
    def kept(l):
        return -(-l // T)                      # ceil(l / T)
    first = all(l * t_attn + l * t_ffn + 2 * l * t_ar >= (l - kept(l)) * tau_ffn + l * tau_attn
                for l in range(1, L + 1))
    second = all(l * t_attn + (l - 1) * t_ffn + (2 * l - 1) * t_ar >= (l - kept(l)) * tau_ffn + (l - 1) * tau_attn
                 for l in range(1, L + 1))
    return first and second
