"""Each pin is only worth something if a plausible mistake in the oracle fails it.  This file plants
such mistakes in a COPY of the oracle on the CPU (one patched line of the C source built into a
temporary library, or one patched line of a Python composition) and checks that the named pin
raises.  Nothing here touches the oracle that the parity tests use."""
import ctypes as C
import inspect
import os
import subprocess
import textwrap

import numpy as np
import pytest

import oracle as oracle_pkg
from oracle import Oracle

import test_oracle_pins as pins

SRC = os.path.join(os.path.dirname(oracle_pkg.__file__), "alora_oracle.c")


class _PatchedOracle(Oracle):
    """The f64 oracle built from the C source with `old` replaced by `new` (exactly one occurrence)."""

    def __init__(self, tmp_path, old: str, new: str):
        text = open(SRC).read()
        assert text.count(old) == 1, (old, text.count(old))
        c = tmp_path / "mutant.c"
        so = tmp_path / "mutant.so"
        c.write_text(text.replace(old, new))
        subprocess.check_call(["gcc", "-O1", "-fopenmp", "-shared", "-fPIC", "-DORACLE_REAL=double", "-o", str(so),
                               str(c), "-lm"])
        self.precision = "f64"
        self.lib = C.CDLL(str(so))
        self.lib.oracle_real_bytes.restype = C.c_int


# (source line as it stands, the planted mistake, pins that must notice)
C_MUTANTS = [
    ("gate = force_all ? 1 : (positions[t] >= activation_offsets[r]);",
     "gate = force_all ? 1 : (positions[t] > activation_offsets[r]);",
     ["test_projection_matches_library_matmul", "test_hand_example_eq5"]),
    ("const int g = h / G; /* KV head shared by this group of query heads */",
     "const int g = h % Hkv;",
     ["test_group_head_mapping_brute_force", "test_attention_matches_library_sdpa:4:2"]),
    ("yt[first[b] + n] = (double)((real)yt[first[b] + n] + s * d);",
     "yt[first[b] + n] = (double)((real)yt[first[b] + n] + d);",
     ["test_projection_matches_library_matmul"]),
    ("const int nk = p + 1; /* keys 0..p visible */",
     "const int nk = p > 0 ? p : 1;",
     ["test_attention_matches_library_sdpa:4:2", "test_attention_closed_forms"]),
    ("s *= (real)softmax_scale;",
     "",
     ["test_attention_matches_library_sdpa:4:2", "test_attention_closed_forms"]),
    ("for (int i = 0; i < rk; ++i) d += (real)Bs[b][(size_t)n * rk + i] * u[i];",
     "for (int i = 0; i < rk; ++i) d += (real)Bs[b][(size_t)i * width[b] + n] * u[i];",
     ["test_projection_matches_library_matmul", "test_full_activation_is_merged_weight_lora"]),
    ("w[j] = (real)exp((double)(w[j] - m));",
     "w[j] = (real)exp((double)(w[j]));",
     ["test_attention_closed_forms"]),
    ("slots[t] = (int64_t)block_tables[(size_t)r * max_blocks + blk] * page_size + p % page_size;",
     "slots[t] = (int64_t)block_tables[(size_t)r * max_blocks + blk] * page_size + (p + 1) % page_size;",
     ["test_slot_mapping_brute_force_and_page_permutation", "test_pool_layout_by_plain_indexing"]),
    ("const real inv = (real)1 / (real)sqrt((double)(ss / (real)H + (real)eps));",
     "const real inv = (real)1 / (real)sqrt((double)(ss + (real)eps));",
     ["test_rmsnorm_swiglu_linear_against_library", "test_decoder_layer_against_library_restatement"]),
    # the cache layout: planes and heads exchanged consistently in append and gather
    ("return ((((size_t)page * 2 + (size_t)plane) * Hkv + (size_t)head) * page_size + (size_t)row) * hd;",
     "return ((((size_t)page * Hkv + (size_t)head) * 2 + (size_t)plane) * page_size + (size_t)row) * hd;",
     ["test_pool_layout_by_plain_indexing"]),
    # rows and heads exchanged inside a plane
    ("return ((((size_t)page * 2 + (size_t)plane) * Hkv + (size_t)head) * page_size + (size_t)row) * hd;",
     "return ((((size_t)page * 2 + (size_t)plane) * page_size + (size_t)row) * Hkv + (size_t)head) * hd;",
     ["test_pool_layout_by_plain_indexing"]),
    # rotary embedding: neighbouring columns paired instead of the two halves of the head
    ("const real lo = (real)v[i], hi = (real)v[i + half];\n                v[i] = (double)(lo * c - hi * s);\n                v[i + half] = (double)(hi * c + lo * s);",
     "const real lo = (real)v[2 * i], hi = (real)v[2 * i + 1];\n                v[2 * i] = (double)(lo * c - hi * s);\n                v[2 * i + 1] = (double)(hi * c + lo * s);",
     ["test_rope_against_complex_multiplication_and_hand_example"]),
    # ... the rotation turned the other way
    ("v[i] = (double)(lo * c - hi * s);", "v[i] = (double)(lo * c + hi * s);",
     ["test_rope_against_complex_multiplication_and_hand_example", "test_rope_scores_depend_on_the_position_difference_only"]),
    # ... the frequency exponent without its factor two
    ("const double a = (double)positions[t] * pow(theta, -2.0 * (double)i / (double)hd);",
     "const double a = (double)positions[t] * pow(theta, -1.0 * (double)i / (double)hd);",
     ["test_rope_against_complex_multiplication_and_hand_example"]),
    ("const real u = (real)gate_up[(size_t)t * 2 * I + I + i];",
     "const real u = (real)gate_up[(size_t)t * 2 * I + i]; (void)I;",
     ["test_rmsnorm_swiglu_linear_against_library", "test_decoder_layer_against_library_restatement"]),
    # the gated MLP matrix: gate one position late, scale dropped, B read transposed
    ("gate = force_all || positions[t] >= activation_offsets[r];   /* the MLP gate */",
     "gate = force_all || positions[t] > activation_offsets[r];",
     ["test_mlp_gated_linear_special_cases", "test_decoder_layer_with_mlp_adapters_against_library_restatement"]),
    ("yt[n] = (double)((real)yt[n] + s * d);   /* MLP delta add */",
     "yt[n] = (double)((real)yt[n] + d); (void)s;",
     ["test_mlp_gated_linear_special_cases", "test_decoder_layer_with_mlp_adapters_against_library_restatement"]),
    ("d += (real)B[k][(size_t)n * rk + i] * u[i];   /* MLP expand */",
     "d += (real)B[k][(size_t)i * N + n] * u[i];",
     ["test_mlp_gated_linear_special_cases"]),
]


def _run_pin(name: str, orc):
    fn_name, *params = name.split(":")
    fn = getattr(pins, fn_name)
    sig = inspect.signature(fn)
    kwargs = {}
    for p in sig.parameters:
        if p in ("oracle64", "oracle32"):
            kwargs[p] = orc
    if params:
        kwargs["Hq"], kwargs["Hkv"] = int(params[0]), int(params[1])
    fn(**kwargs)


@pytest.mark.parametrize("idx", range(len(C_MUTANTS)))
def test_planted_mistake_in_the_c_oracle_fails_its_pins(tmp_path, idx):
    old, new, must_fail = C_MUTANTS[idx]
    mutant = _PatchedOracle(tmp_path, old, new)
    for name in must_fail:
        with pytest.raises(AssertionError):
            _run_pin(name, mutant)


PY_MUTANTS = [
    # the MLP residual taken from the layer input instead of the post-attention state
    ('h2 = h1 + self.linear(self.swiglu(self.linear(xm, lw["wgate_up"])), lw["wdown"])',
     'h2 = _f64(h) + self.linear(self.swiglu(self.linear(xm, lw["wgate_up"])), lw["wdown"])'),
    # the two norm gains exchanged
    ('xn = self.rmsnorm(h, lw["norm_attn"], eps)', 'xn = self.rmsnorm(h, lw["norm_mlp"], eps)'),
    ('xm = self.rmsnorm(h1, lw["norm_mlp"], eps)', 'xm = self.rmsnorm(h1, lw["norm_attn"], eps)'),
    # post-norm instead of pre-norm on the MLP branch
    ('xm = self.rmsnorm(h1, lw["norm_mlp"], eps)', 'xm = h1'),
    # attention residual dropped
    ('h1 = _f64(h) + self.linear(blk["out"], lw["wo"])', 'h1 = self.linear(blk["out"], lw["wo"])'),
    # adapted MLP: the up projection given the gate projection's pair, the down pair applied to the normed input's
    # width-compatible sibling (the gate pair's B is [I, r], so the down projection's pair must be its own), the MLP
    # gate left open, the adapted down projection fed the un-activated gate output
    ('up = gated(xm, lw["wgate_up"][inter:], "Au", "Bu")', 'up = gated(xm, lw["wgate_up"][inter:], "Ag", "Bg")',
     "test_decoder_layer_with_mlp_adapters_against_library_restatement"),
    ('gate = gated(xm, lw["wgate_up"][:inter], "Ag", "Bg")', 'gate = gated(xm, lw["wgate_up"][:inter], "Au", "Bu")',
     "test_decoder_layer_with_mlp_adapters_against_library_restatement"),
    ("[getattr(m, a) for m in mlp_adapters], [getattr(m, b) for m in mlp_adapters], force_all)",
     "[getattr(m, a) for m in mlp_adapters], [getattr(m, b) for m in mlp_adapters], True)",
     "test_cache_reuse_identity_through_two_layers_with_mlp_adapters"),
    ('h2 = h1 + gated(act, lw["wdown"], "Ad", "Bd")', 'h2 = h1 + self.linear(act, lw["wdown"])',
     "test_decoder_layer_with_mlp_adapters_against_library_restatement"),
    ('act = self.swiglu(np.concatenate([gate, up], axis=1))', 'act = self.swiglu(np.concatenate([up, gate], axis=1))',
     "test_decoder_layer_with_mlp_adapters_against_library_restatement"),
]


@pytest.mark.parametrize("idx", range(len(PY_MUTANTS)))
def test_planted_mistake_in_the_layer_composition_fails_its_pin(oracle64, idx):
    old, new, *pin = PY_MUTANTS[idx]
    pin_fn = getattr(pins, pin[0] if pin else "test_decoder_layer_against_library_restatement")
    src = textwrap.dedent(inspect.getsource(Oracle.decoder_layer))
    assert src.count(old) == 1, old
    ns = dict(vars(oracle_pkg))
    exec(src.replace(old, new), ns)

    class Mutant(Oracle):
        decoder_layer = ns["decoder_layer"]

        def __init__(self, base):
            self.precision, self.lib = base.precision, base.lib

    with pytest.raises(AssertionError):
        pin_fn(Mutant(oracle64))
    # and the unpatched composition passes the same call
    pin_fn(oracle64)
