"""Are the pins sharp?  Each case plants one plausible mistake in a copy of the oracle (on the CPU:
a mutated pec_oracle.c compiled to a scratch library, or a mutated copy of reference.py) and checks
that at least one pin test fails.  The real oracle is never touched."""
import ctypes
import importlib.util
import os
import subprocess
import sys
import types

import pytest

import oracle
import oracle.reference as ref
import test_oracle_pins as pins
import test_oracle_planner as plan_pins
import test_sp_cost_model as sp_pins
import test_ring_and_batches as ring_pins
import test_worklist_planner as wl_pins

HERE = os.path.dirname(os.path.abspath(__file__))
ORACLE_DIR = os.path.join(os.path.dirname(HERE), "oracle")


def _expand(fn):
    """All parametrised invocations of a test function as zero-argument callables."""
    calls = []
    marks = [m for m in getattr(fn, "pytestmark", []) if m.name == "parametrize"]
    if not marks:
        return [fn]
    def rec(i, kwargs):
        if i == len(marks):
            calls.append(lambda kw=dict(kwargs): fn(**kw))
            return
        names = [n.strip() for n in marks[i].args[0].split(",")]
        for val in marks[i].args[1]:
            vals = val if len(names) > 1 else (val,)
            rec(i + 1, {**kwargs, **dict(zip(names, vals))})
    rec(0, {})
    return calls


def _pin_calls(module):
    out = []
    for name in sorted(dir(module)):
        if name.startswith("test_"):
            out += _expand(getattr(module, name))
    return out


def _some_pin_fails(calls):
    for call in calls:
        try:
            call()
        except AssertionError:
            return True
        except Exception:            # a crash inside a pin (NaN, shape error) also exposes the mistake
            return True
    return False


def _all_oracle_pins():
    # of the cost-model tests only the two that pin the oracle itself (the others compare the library with it)
    return (_pin_calls(pins) + _pin_calls(plan_pins) +
            [sp_pins.test_oracle_volumes_match_the_hand_worked_example, sp_pins.test_oracle_limiting_cases] +
            _pin_calls(ring_pins) +
            _expand(wl_pins.test_worklist_covers_every_row_once_heaviest_first) + _expand(wl_pins.test_partition_rows_split_the_chunk) +
            [wl_pins.test_worklist_hand_worked_example, wl_pins.test_worklist_ties_keep_request_then_position_order])


def test_the_unmutated_oracle_passes_every_pin():
    assert not _some_pin_fails(_all_oracle_pins())


C_MUTATIONS = {
    "scale dropped": ("a[n] = s * scale;", "a[n] = s;"),
    "causal limit exclusive": ("if (causal && j > q_pos[r]) continue;", "if (causal && j >= q_pos[r]) continue;"),
    "causal mask ignored": ("if (causal && j > q_pos[r]) continue;", ""),
    "GQA head mapping by modulo": ("const int kvh = h / group;", "const int kvh = h % hkv;"),
    "scores use V instead of K": ("const float *kr = k + ((size_t)j * hkv + kvh) * d;", "const float *kr = v + ((size_t)j * hkv + kvh) * d;"),
    "sign of the max in the row sum": ("l += exp(a[t] - m);", "l += exp(a[t] + m);"),
    "LSE without the max": ("lse[(size_t)r * hq + h] = m + log(l);", "lse[(size_t)r * hq + h] = log(l);"),
    "normalisation dropped": ("const double p = exp(a[t] - m) / l;", "const double p = exp(a[t] - m);"),
    "value row by visible index instead of key index": ("(size_t)idx[t] * hkv", "(size_t)t * hkv"),
    "first key of an interval dropped": ("for (int64_t j = iv_lo[t]; j < iv_hi[t]; ++j) {", "for (int64_t j = iv_lo[t] + 1; j < iv_hi[t]; ++j) {"),
    "empty row LSE zero": ("lse[(size_t)r * hq + h] = -INFINITY;", "lse[(size_t)r * hq + h] = 0.0;"),
    "query head offset dropped": ("const float *qr = q + ((size_t)r * hq + h) * d;", "const float *qr = q + ((size_t)r * hq) * d;"),
    "output weighted by unnormalised value channel order": ("orow[c] += p * (double)vr[c];", "orow[c] += p * (double)vr[d - 1 - c];"),
}


@pytest.mark.parametrize("name", sorted(C_MUTATIONS))
def test_a_mistake_in_the_attention_oracle_is_caught(name, tmp_path, monkeypatch):
    old, new = C_MUTATIONS[name]
    src = open(os.path.join(ORACLE_DIR, "pec_oracle.c")).read()
    assert src.count(old) == 1, f"mutation site not unique: {old}"
    mutant_c = tmp_path / "mutant.c"
    mutant_c.write_text(src.replace(old, new))
    lib_path = tmp_path / "libmutant.so"
    subprocess.run(["gcc", "-O2", "-fPIC", "-shared", "-fopenmp", "-std=c11", "-o", str(lib_path), str(mutant_c), "-lm"], check=True)
    real = ref._load()
    lib = ctypes.CDLL(str(lib_path))
    lib.pec_oracle_attn_rows.restype = real.pec_oracle_attn_rows.restype
    lib.pec_oracle_attn_rows.argtypes = real.pec_oracle_attn_rows.argtypes
    lib.pec_oracle_threads.restype = ctypes.c_int
    monkeypatch.setattr(ref, "_lib", lib)
    assert _some_pin_fails(_pin_calls(pins)), f"no pin noticed: {name}"


PY_MUTATIONS = {
    "zigzag pairs block p with block 2P-p": ("(bounds[2 * P - 1 - p], bounds[2 * P - p])", "(bounds[2 * P - p - 1 - (p > 0)], bounds[2 * P - p - (p > 0)])"),
    "bounds not clamped to S": ("bounds = [min(S, align * ((k * U) // (2 * P)))", "bounds = [(align * ((k * U) // (2 * P)))"),
    "pairs count S-j-1": ("n += (S - j) if causal else S", "n += (S - j - 1) if causal else S"),
    "tile SKIP test off by one": ("elif k0 > q1 - 1:", "elif k0 > q1:"),
    "tile FULL test off by one": ("elif k1 - 1 <= q0:", "elif k1 <= q0:"),
    "last chunk not cut": ("chunks = [(c * C, min(S, (c + 1) * C) - c * C)", "chunks = [(c * C, C)"),
    "merge weights swapped": ("o = ca[..., None] * o_a + cb[..., None] * o_b", "o = cb[..., None] * o_a + ca[..., None] * o_b"),
    "merge LSE without log": ("m_safe + np.log(np.where(both_empty, 1.0, tot)))\n    ca", "m_safe + (np.where(both_empty, 1.0, tot)))\n    ca"),
    "merge_n forgets the max shift": ("lse = np.where(empty, -np.inf, m_safe + np.log(np.where(empty, 1.0, tot)))", "lse = np.where(empty, -np.inf, np.log(np.where(empty, 1.0, tot)))"),
    "kv prefix ignored": ("        hi = min(hi, kv_len)\n", ""),
    "Megatron attention term not divided by T": ("qkv / T + 4 * (s * T) ** 2 * d / T + out_proj", "qkv / T + 4 * (s * T) ** 2 * d + out_proj"),
    "Ulysses all-to-all counts G not G-1": ("a2a = 2 * s * (n_h + n_kv) * d_h * (G - 1)", "a2a = 2 * s * (n_h + n_kv) * d_h * G"),
    "linear without the transpose of w": ('@ _as_f32(w).astype(np.float64).T', '@ _as_f32(w).astype(np.float64)[:, ::-1].T'),
    "ring sends the keys the other way round": ("keys = seg[(r - t) % P]", "keys = seg[(r + t) % P]"),
    "ring step forgets the diagonal key": ("last = min(k_hi, i + 1) if causal else k_hi", "last = min(k_hi, i) if causal else k_hi"),
    "contiguous segments cut like zigzag blocks": ("b = [min(S, align * ((k * U) // P)) for k in range(P + 1)]", "b = [min(S, align * ((k * U) // (2 * P))) for k in range(P + 1)]"),
    "batches built shortest first": ("longest = max(lengths[i] for i in remaining)", "longest = min(lengths[i] for i in remaining)"),
    "batch goes to the fullest replica": ("rep = tokens.index(min(tokens))", "rep = tokens.index(max(tokens))"),
    "work-list weight from the tile's first row": ("weight = _ceil_div(pos0 + n if causal else L, block_n)", "weight = _ceil_div(pos0 + 1 if causal else L, block_n)"),
    "work-list lightest first": ("entries.append((-weight, b, pos0, (cu[b], pos0, n, L)))", "entries.append((weight, b, pos0, (cu[b], pos0, n, L)))"),
    "work-list ties by position before request": ("entries.sort(key=lambda e: e[:3])", "entries.sort(key=lambda e: (e[0], e[2], e[1]))"),
    "work-list last tile not cut": ("n = min(block_m, L - pos0)", "n = block_m"),
    "partition rows ignore the chunk start": ("range(max(lo, chunk_start), min(hi, chunk_start + chunk_len))", "range(lo, min(hi, chunk_start + chunk_len))"),
    "rope turns the other way": ("out[:, h0:h0 + half] = a * c - b * s_", "out[:, h0:h0 + half] = a * c + b * s_"),
    "rope second half without the cross term": ("out[:, h0 + half:h0 + head_dim] = b * c + a * s_", "out[:, h0 + half:h0 + head_dim] = b * c"),
    "rope frequency exponent i/d": ("** (-2.0 * np.arange(half, dtype=np.float64) / head_dim)", "** (-1.0 * np.arange(half, dtype=np.float64) / head_dim)"),
    "rope pairs neighbouring channels": ("        a = out[:, h0:h0 + half].copy()\n        b = out[:, h0 + half:h0 + head_dim].copy()\n        out[:, h0:h0 + half] = a * c - b * s_\n        out[:, h0 + half:h0 + head_dim] = b * c + a * s_",
                                         "        a = out[:, h0:h0 + head_dim:2].copy()\n        b = out[:, h0 + 1:h0 + head_dim:2].copy()\n        out[:, h0:h0 + head_dim:2] = a * c - b * s_\n        out[:, h0 + 1:h0 + head_dim:2] = b * c + a * s_"),
    "rope turns the values too": ("for h0 in range(0, rot_cols, head_dim):", "for h0 in range(0, out.shape[1], head_dim):"),
    "rope angle from the row index": ("ang = pos[:, None] * inv_freq[None, :]", "ang = np.arange(len(pos), dtype=np.float64)[:, None] * inv_freq[None, :]"),
    "MLP parameter volume 4 d^2": ("(8 * d * d * (T - 1) * G / T, 16 * s * d * d)", "(4 * d * d * (T - 1) * G / T, 16 * s * d * d)"),
}


@pytest.mark.parametrize("name", sorted(PY_MUTATIONS))
def test_a_mistake_in_the_python_oracle_is_caught(name, monkeypatch):
    old, new = PY_MUTATIONS[name]
    src = open(os.path.join(ORACLE_DIR, "reference.py")).read()
    assert src.count(old) == 1, f"mutation site not unique: {old}"
    mod = types.ModuleType("oracle.reference_mutant")
    mod.__package__ = "oracle"
    mod.__file__ = ref.__file__
    exec(compile(src.replace(old, new), "reference_mutant.py", "exec"), mod.__dict__)
    for attr in ("attn_rows", "prefill_attn", "varlen_attn", "merge", "merge_n", "plan_partitions",
                 "partition_intervals", "sp_volumes", "select_sp", "linear", "plan_ring", "ring_segments",
                 "balance_batches", "plan_worklist", "partition_rows", "rope", "linear_rope"):
        monkeypatch.setattr(oracle, attr, getattr(mod, attr))
    # The ring/batch pin file also compares the library with the oracle; here the library is replaced by an
    # echo of the mutant, so that only the pins proper (enumeration, hand-worked values, bounds) can object.
    names = {v: k for k, v in ring_pins.LAYOUTS.items()}
    echo = types.SimpleNamespace(
        pec_plan_ring=lambda S, P, align=128, layout=0, causal=True: mod.plan_ring(S, P, align, names[layout], causal),
        pec_balance_batches=lambda lengths, replicas: mod.balance_batches(lengths, replicas),
        PecError=ValueError, PEC_LAYOUT_ZIGZAG=0, PEC_LAYOUT_CONTIGUOUS=1)
    monkeypatch.setattr(ring_pins, "binding", echo)
    assert _some_pin_fails(_all_oracle_pins()), f"no pin noticed: {name}"
