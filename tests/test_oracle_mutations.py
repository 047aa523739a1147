"""Do the pins hold the oracle?  Every case below plants one plausible mistake in a copy of the oracle's
source (a dropped term, a wrong sign, constant or index, the wrong operand), runs the pin tests of
test_oracle_formats / test_oracle_quantizer / test_oracle_attention against that copy and demands that at
least one of them fails -- not counting the pins that compare the oracle with a second implementation of the same
formulas, so that every mistake is caught by something the paper or the mathematics fixes (a closed form, a
library routine, an invariant, a special case, an error bound).  Everything runs on the CPU; the oracle on disk
is never touched."""
import inspect
import pathlib
import sys
import types

import pytest

from tests import test_oracle_attention, test_oracle_formats, test_oracle_quantizer

PIN_MODULES = (test_oracle_formats, test_oracle_quantizer, test_oracle_attention)
SOURCE = (pathlib.Path(__file__).resolve().parents[1] / "oracle" / "kvq_oracle.py").read_text()

# (what the mistake is, text in the oracle, what it becomes[, how many places])
MUTATIONS = [
    # ---- number formats
    ("E4M3 exponent bias 8 in the decoder", "np.exp2((e - 7).astype(np.float64))", "np.exp2((e - 8).astype(np.float64))"),
    ("E4M3 subnormals decoded as zero", "sub = (m / 8.0) * 2.0 ** -6", "sub = 0.0 * m"),
    ("E4M3 encoder truncates instead of rounding", "q = np.rint(v / ulp) * ulp", "q = np.floor(v / ulp) * ulp"),
    ("E4M3 step not floored at 2^-9", "q = np.clip(q, 2.0 ** -9, 448.0)", "q = np.clip(q, 0.0, 448.0)"),
    ("BF16 conversion truncates", "r = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)", "r = u >> np.uint32(16)"),
    # ---- rotation
    ("rotation not normalised", "    return y / math.sqrt(d)", "    return y"),
    ("butterfly outputs swapped", "np.stack([rounder(a + b), rounder(a - b)], axis=-2)", "np.stack([rounder(a - b), rounder(a + b)], axis=-2)"),
    ("c_128 = 2^-3", "128: float(np.float32(2.0 ** -3.5))", "128: float(np.float32(2.0 ** -3.0))"),
    ("binary32 rotation skips the final scaling", "    return f32(y * C_D[d])", "    return f32(y)"),
    ("binary32 rotation rounds only at the end", "    y = _butterflies(x, d, f32)\n", "    y = _butterflies(x, d, lambda t: t)\n"),
    # ---- quantizer
    ("2^b levels instead of 2^b - 1", "L = float(2 ** bits - 1)", "L = float(2 ** bits)"),
    ("zero-point with the wrong sign", "z = -np.rint(rnd(mn / ds))", "z = np.rint(rnd(mn / ds))"),
    ("zero-point from the maximum", "z = -np.rint(rnd(mn / ds))", "z = -np.rint(rnd(mx / ds))"),
    ("zero-point from the unrounded step", "z = -np.rint(rnd(mn / ds))", "z = -np.rint(rnd(mn / np.maximum(step, 2.0 ** -9)))"),
    ("codes without the zero-point", "c = np.rint(rnd(yg / ds[..., None])) + zs[..., None]", "c = np.rint(rnd(yg / ds[..., None]))"),
    ("codes truncated instead of rounded", "c = np.rint(rnd(yg / ds[..., None]))", "c = np.floor(rnd(yg / ds[..., None]))"),
    ("codes not clamped", "c = np.clip(c, 0.0, L)", "c = c + 0.0"),
    ("groups interleaved instead of consecutive", "yg = y.reshape(y.shape[:-1] + (G, group))",
     "yg = np.swapaxes(y.reshape(y.shape[:-1] + (group, G)), -1, -2)"),
    ("packing with element 0 in the most significant bits", "np.uint8(i * bits)", "np.uint8((per - 1 - i) * bits)", 2),
    ("keys stored unrotated", "    if cache.rotate_k:\n        k = rotate_f32_steps(k, cache.signs)", "    if False:\n        k = rotate_f32_steps(k, cache.signs)"),
    ("values rotated by default", "    if cache.rotate_v:\n        v = rotate_f32_steps", "    if cache.rotate_k:\n        v = rotate_f32_steps"),
    ("value metadata written to the key arrays", "    cache.v_scale[:, :, sl] = vs", "    cache.k_scale[:, :, sl] = vs"),
    ("ring slots not wrapped", "            return idx % self.capacity", "            return idx"),
    # ---- reconstruction and attention
    ("reconstruction adds the zero-point", "((cg - zs[..., None]) * ds[..., None])", "((cg + zs[..., None]) * ds[..., None])"),
    ("bias added instead of subtracted", "s_s = s_s - b ", "s_s = s_s + b "),
    ("bias also taken off the current scores", "    s = np.concatenate([s_s, s_r], axis=1)",
     "    s = np.concatenate([s_s, s_r - (b.mean() if (n_s > 0 and correction) else 0.0)], axis=1)"),
    ("1/12 instead of 1/24", "(sigma * sigma / 24.0)", "(sigma * sigma / 12.0)"),
    ("softmax scale not squared in the bias", "(sigma * sigma / 24.0)", "(sigma / 24.0)"),
    ("step not squared in the bias", "(nu @ (key_scale ** 2).T)", "(nu @ key_scale.T)"),
    ("group norms without the square", "nu = (q_rot.reshape(q.shape[0], G, k_group) ** 2).sum(axis=-1)",
     "nu = np.abs(q_rot.reshape(q.shape[0], G, k_group)).sum(axis=-1)"),
    ("group norms of the unrotated query", "nu = (q_rot.reshape(", "nu = (q.reshape("),
    ("bias from the value steps", "ds = e4m3_decode(k_scale)\n            b =", "ds = e4m3_decode(v_scale)\n            b ="),
    ("cached scores from the unrotated query", "s_s = sigma * (q_rot @ k_hat.T)", "s_s = sigma * (q @ k_hat.T)"),
    ("current scores without the softmax scale", "s_r = sigma * (q @ kr.T)", "s_r = q @ kr.T"),
    ("current scores from the rotated query", "s_r = sigma * (q @ kr.T)", "s_r = sigma * (q_rot @ kr.T)"),
    ("exact bias with alpha twice too large", "a = 0.5 * sigma * q_rot[:, None, :]", "a = sigma * q_rot[:, None, :]"),
    ("log sinhc series with a wrong sign", "a2 / 6.0 - a2 ** 2 / 180.0", "a2 / 6.0 + a2 ** 2 / 180.0"),
    ("log sinhc for large arguments without the log term", "a[big] - np.log(2.0 * a[big])", "a[big]"),
    ("log-sum-exp without the maximum", '"lse": (mx + np.log(z))[:, 0]', '"lse": (np.log(z))[:, 0]'),
    ("cached mass taken over the current keys", '"cached_mass": p[:, :n_s].sum(axis=1)', '"cached_mass": p[:, n_s:].sum(axis=1)'),
    ("output without the current chunk's values", "out = o_s + p[:, n_s:] @ vr", "out = o_s"),
    ("rotated values not rotated back", "        o_s = rotate_f64(o_s, None)\n", "        o_s = o_s + 0.0\n"),
    ("per-channel keys take the token's own row of steps", "ksl = sl // cache.group if cache.k_per_channel else sl",
     "ksl = sl % (cache.capacity // cache.group) if cache.k_per_channel else sl"),
    # ---- attention-weight diagnostics
    ("JSD without the halves", "return 0.5 * kl(p) + 0.5 * kl(r)", "return kl(p) + kl(r)"),
    ("JSD one-sided", "return 0.5 * kl(p) + 0.5 * kl(r)", "return 0.5 * kl(p) + 0.5 * kl(p)"),
    ("JSD mixture not halved", "m = 0.5 * (p + r)", "m = p + r"),
    ("BF16 reference weights without the softmax scale", "s = sigma * (q @ bf16_bits_to_f64(k_bits).T)", "s = q @ bf16_bits_to_f64(k_bits).T"),
    ("JSD reference keys in the wrong order", "k_all = np.concatenate([kcached_bits[b, h], kcur_bits[b, h]], axis=0)",
     "k_all = np.concatenate([kcur_bits[b, h], kcached_bits[b, h]], axis=0)"),
    ("weights returned unnormalised", '        res["weights"] = p', '        res["weights"] = e'),
    ("JSD of the uncorrected weights only", "cache.bits, cache.group, sigma, correction, cache.rotate_k, cache.signs, rows,\n            return_weights=True)",
     "cache.bits, cache.group, sigma, False, cache.rotate_k, cache.signs, rows,\n            return_weights=True)"),
    ("effective bits count 16 metadata bits", "return bits + 24.0 / group", "return bits + 16.0 / group"),
]


def _mutant(old, new, count=1):
    assert SOURCE.count(old) == count, f"the oracle no longer contains {old!r} exactly {count} time(s)"
    mod = types.ModuleType("kvq_oracle_mutant")
    mod.__dict__["__name__"] = "kvq_oracle_mutant"
    sys.modules["kvq_oracle_mutant"] = mod        # dataclasses look their module up by name
    try:
        exec(compile(SOURCE.replace(old, new), "kvq_oracle_mutant.py", "exec"), mod.__dict__)
    finally:
        del sys.modules["kvq_oracle_mutant"]
    return mod


# pins that retype the method's formulas as scalar loops: useful, but they do not count here
SECOND_IMPLEMENTATIONS = {"test_brute_force_tiny", "test_brute_force_second_implementation",
                          "test_per_channel_keys_against_the_scalar_implementation"}


def _pins():
    for m in PIN_MODULES:
        for name, fn in inspect.getmembers(m, inspect.isfunction):
            if name.startswith("test_") and fn.__module__ == m.__name__ and name not in SECOND_IMPLEMENTATIONS:
                yield m, name, fn


def first_failing_pin(oracle_module):
    """Runs the pins against `oracle_module`; the name of the first one that fails, else None."""
    saved = [(m, m.O) for m in PIN_MODULES]
    try:
        for m in PIN_MODULES:
            m.O = oracle_module
        for m, name, fn in _pins():
            try:
                fn()
            except Exception:            # an assertion, or the mutant breaking down inside the pin
                return name
    finally:
        for m, o in saved:
            m.O = o
    return None


def test_the_unmodified_source_passes_every_pin():
    assert first_failing_pin(_mutant("import math", "import math")) is None


@pytest.mark.parametrize("case", MUTATIONS, ids=[c[0] for c in MUTATIONS])
def test_a_planted_mistake_fails_a_pin(case):
    what, old, new = case[:3]
    killer = first_failing_pin(_mutant(old, new, *case[3:]))
    assert killer is not None, f"no pin notices: {what}"
