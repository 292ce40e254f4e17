"""GPU parity: the CUDA library against the CPU oracle, through the C ABI, on seeded inputs."""
import numpy as np
import pytest

from conftest import gpu_cfg
from paper_2507_23777_b200 import inputs

pytestmark = pytest.mark.gpu

F32_TOL = dict(atol=2e-4, rtol=2e-4)
BF16_TOL = dict(atol=2e-2, rtol=1e-2)     # the stated bound for bf16 storage


@pytest.fixture(scope="module")
def P():
    import torch
    assert torch.cuda.is_available(), "these tests need a B200"
    from paper_2507_23777_b200 import build
    build.build()
    import parity
    return parity


def scripted(ls, full, rng, good):
    """Drafts that make exactly `good[b]` acceptances under strict greedy verification."""
    K, V = ls.K, ls.V
    st = ls.ctx.xsm_debug_get_state()
    dr = np.zeros((ls.B, K), dtype=np.int32)
    for b in range(ls.B):
        n = int(st["len"][b])
        t = full[b][n + 1:n + 1 + K].copy()
        for j in range(good[b], K):
            t[j] = (t[j] + 1 + int(rng.integers(0, V - 1))) % V
        if good[b] < K:
            t[good[b]] = (full[b][n + 1 + good[b]] + 1) % V
        dr[b] = t
    return dr


@pytest.mark.parametrize("dtype,phase_launch,batch", [(0, True, 1), (0, False, 1), (1, False, 1), (0, False, 3), (1, True, 3)])
def test_unit_model_lockstep_with_scripted_accept_lengths(P, dtype, phase_launch, batch):
    """Hand-sized model, ragged shapes (V=50, C=5, dh=32, 32-token pages): every accept length 0..K occurs,
    logits, committed tokens, windows and the cache agree with the oracle; output is plain greedy."""
    # bf16: weights scaled so that logits have the magnitude of the real configurations (about 0.5),
    # which is what the absolute part of the bf16 bound assumes
    cfg = gpu_cfg(dtype=dtype, n_draft=3, sigma=0.15 if dtype == 0 else 0.05)
    tol = F32_TOL if dtype == 0 else BF16_TOL
    ls = P.LockStep(cfg, batch=batch, random_gains=True, phase_launch=phase_launch)
    ls.begin()
    # the greedy continuation of every sequence, from the oracle's independent plain loop
    full = []
    for b in range(batch):
        ref = ls.orc.new_seq(ls.cond[b], b).generate_plain([0], ls.odc, 90)
        full.append(np.concatenate([[0], ref]))
    rng = np.random.default_rng(0)
    outs = [[] for _ in range(batch)]
    seen = set()
    for it in range(14):
        good = [int(rng.integers(0, 4)) for _ in range(batch)]
        toks, acc = ls.step(drafts=scripted(ls, full, rng, good), margin=1e-3 if dtype == 0 else 1e-2, **tol)
        for b in range(batch):
            outs[b].extend(toks[b])
            seen.add(acc[b])
        if ls.excused == 0:
            assert acc == good
    assert seen == {0, 1, 2, 3} or ls.excused > 0
    if ls.excused == 0:
        for b in range(batch):
            assert outs[b] == full[b][1:1 + len(outs[b])].tolist()
    ls.compare_cache(**tol)
    st = ls.ctx.xsm_debug_get_state()
    for b in range(batch):
        assert st["pages"][b] == -(-(st["len"][b] + 4) // 32)
    ls.close()


def test_config0_tiny_fp32_full_run_is_bit_exact(P):
    """Config 0: 512 tokens, K=3, strict greedy: token sequence and accept lengths equal the oracle's."""
    import oracle
    from paper_2507_23777_b200 import binding
    cfg = inputs.config(0)
    w = inputs.make_weights(cfg)
    cond = inputs.make_cond(cfg)
    orc = oracle.Oracle(cfg, w)
    dc = oracle.decode_config(cfg)
    s = orc.new_seq(cond[0], 0)
    s.begin([0], dc)
    ref, ref_steps, ref_hist = s.generate(dc, 512)
    ctx = binding.Context(cfg, w)
    ctx.prefill(cond, [0], binding.decode_config(cfg))
    toks, lens, st = ctx.generate(512)
    assert lens[0] == 512 and np.array_equal(toks[0], ref)
    assert st.steps == ref_steps and list(st.accept_hist)[:4] == ref_hist and st.tokens == 512
    assert abs(st.scr - 512 / ref_steps) < 1e-12
    ctx.xsm_destroy()


def test_config0_lockstep_logits_and_cache(P):
    cfg = inputs.config(0)
    ls = P.LockStep(cfg)
    ls.begin()
    for _ in range(40):
        ls.step(margin=1e-3, **F32_TOL)
    assert ls.excused == 0
    ls.compare_cache(**F32_TOL)
    ls.close()


def test_config1_small_bf16_prefix(P):
    """Config 1 (12 layers, d=768, K=4, greedy): logits within 2e-2 + 1e-2|ref|, decisions identical
    under teacher forcing except at margins below 1e-2, on a prefix of steps."""
    cfg = inputs.config(1)
    ls = P.LockStep(cfg)
    ls.begin()
    for _ in range(24):
        ls.step(**BF16_TOL)
    assert ls.excused <= 3
    ls.compare_cache(layers=[0, 11], **BF16_TOL)
    ls.close()


def test_config2_medium_bf16_prefix(P):
    """Config 2 (24 layers, d=1024, K=4, top-5 acceptance, top-5 / T=0.5 resampling, output projections x4):
    logits within the bf16 bound, decisions identical under teacher forcing except at small margins."""
    cfg = inputs.config(2)
    ls = P.LockStep(cfg)
    ls.begin()
    for _ in range(12):
        ls.step(**BF16_TOL)
    assert ls.excused <= 3
    ls.compare_cache(layers=[0, 23], **BF16_TOL)
    ls.close()


def test_config2_k0_baseline_path(P):
    """Config 2 with n_draft = 0 (the non-speculative baseline of the same library): one token per step."""
    cfg = inputs.config(2, n_draft=0)
    ls = P.LockStep(cfg)
    ls.begin()
    for _ in range(6):
        _, acc = ls.step(**BF16_TOL)
        assert acc == [0]
    ls.close()


def test_config3_batched_bf16_prefix(P):
    """Config 3: 16 meshes with their own condition and Philox stream in one paged pool, ragged accept lengths."""
    cfg = inputs.config(3)
    ls = P.LockStep(cfg, batch=16)
    ls.begin()
    for _ in range(3):
        ls.step(**BF16_TOL)
    assert ls.excused <= 4
    ls.compare_cache(layers=[11], **BF16_TOL)
    ls.close()


def test_config4_large_bf16_prefix(P):
    """Config 4: 32 layers, d=2048, heads of 128, K=6, batch 4, top-8 acceptance at T=0.7."""
    cfg = inputs.config(4)
    ls = P.LockStep(cfg, batch=4)
    ls.begin()
    for _ in range(2):
        ls.step(**BF16_TOL)
    assert ls.excused <= 2
    ls.close()


@pytest.mark.parametrize("shape", ["heads of 64", "heads of 128, batch 2"])
def test_long_context_split_attention(P, shape):
    """Contexts of many pages: self-attention is split over several CTAs per head and merged (6 and 4 splits
    here), on two-layer models with the widths of configurations 2 and 4.  The oracle is teacher-forced through
    the whole run; logits and the cache are compared at the end, decisions at every step."""
    if shape == "heads of 64":
        cfg, batch, steps = inputs.config(2, n_layers=2, max_seq_len=2048), 1, 300
    else:
        cfg, batch, steps = inputs.config(4, n_layers=2, d_ff=2048, max_seq_len=2048, n_draft=3, n_cond=70), 2, 260
    ls = P.LockStep(cfg, batch=batch)
    ls.begin()
    for it in range(steps):
        ls.step(check_logits=it >= steps - 3, **BF16_TOL)
    st = ls.ctx.xsm_debug_get_state()
    assert st["len"].min() >= steps and ls.excused <= max(3, batch * steps // 20)
    ls.compare_cache(layers=[1], **BF16_TOL)
    ls.close()


def _shape(d, H, dh, f, K, L=2, V=1500, C=40, max_seq_len=256, **kw):
    return dict(d_model=d, n_heads=H, d_head=dh, d_ff=f, d_cond=d, head_hidden=d, n_draft=K, n_layers=L, vocab=V,
                n_cond=C, max_seq_len=max_seq_len, **kw)


SHAPES = {
    "rows of 16 KB, two token rows": (_shape(2048, 16, 128, 8192, 1, L=1, V=1000), 1),
    "sixteen token rows, heads of 32": (_shape(512, 16, 32, 1024, 15, V=777, C=33, page_size=32), 1),
    "fifteen token rows": (_shape(1024, 16, 64, 4096, 4), 3),
    "thirty-two token rows": (_shape(1024, 16, 64, 4096, 7, L=1), 4),
    "forty token rows": (_shape(1024, 16, 64, 4096, 4, L=1), 8),
    "a hundred and twenty token rows": (_shape(1024, 16, 64, 4096, 4, L=1), 24),
    "rows of 3 KB and 12 KB": (_shape(1536, 12, 128, 6144, 2), 2),
    "rows of 1280 and 3840 bytes": (_shape(640, 10, 64, 1920, 3), 1),
    "no heads, five sequences": (_shape(768, 12, 64, 3072, 0), 5),
    "several tile groups per projection": (_shape(2048, 16, 128, 2048, 3, V=3000), 2),
    "two attention items per CTA, pages owned by warps": (_shape(1024, 16, 64, 4096, 0), 16),
    "two attention items per CTA, three token rows each": (_shape(512, 8, 64, 2048, 2, V=900), 24),
    "eight token rows of one sequence (all eight query columns of the transposed attention unit)": (_shape(1024, 16, 64, 4096, 7), 1),
    "six token rows of one sequence, heads of 128": (_shape(1024, 8, 128, 2048, 5, V=1200), 1),
}


@pytest.mark.parametrize("shape", list(SHAPES))
def test_shape_sweep_bf16(P, shape):
    """Shapes between the five configurations: each makes the projections pick another tiling (rows per ring
    item, tiles per group, token tiles, activation chunks).  Three steps, logits and cache against the oracle."""
    ov, batch = SHAPES[shape]
    ls = P.LockStep(inputs.config(2, **ov), batch=batch)
    ls.begin()
    for _ in range(3):
        ls.step(**BF16_TOL)
    ls.compare_cache(**BF16_TOL)
    ls.close()


def test_long_prompt_many_pages_per_attention_split(P):
    """64 heads leave two key splits per head, so at a context of 1100 tokens a split walks nine cache pages and a warp
    owns more than one of them.  The prompt is ingested through the same step kernel; then logits, decisions and the
    whole cache of the last layer are compared with the oracle."""
    cfg = inputs.config(2, **_shape(2048, 64, 32, 2048, 4, max_seq_len=1400))
    cfg["max_seq_len"] = 1400
    ls = P.LockStep(cfg, batch=1)
    prompt = [0] + [int(t) for t in np.random.default_rng(5).integers(1, cfg["vocab"], 1100)]
    st = ls.begin(prompt)
    assert st["len"][0] == len(prompt) - 1
    for _ in range(8):
        ls.step(**BF16_TOL)
    ls.compare_cache(layers=[1], **BF16_TOL)
    ls.close()


def test_sampling_modes_lockstep(P):
    """Top-k acceptance with top-k / temperature resampling and threshold acceptance on the unit model."""
    for over in (dict(verify_mode=1, k_accept=3, sample_mode=1, k_sample=4, temperature=0.7, sigma=0.3),
                 dict(verify_mode=2, delta=0.05, sample_mode=1, k_sample=5, temperature=1.0, sigma=0.3)):
        cfg = gpu_cfg(dtype=0, n_draft=2, seed=5, **over)
        ls = P.LockStep(cfg, batch=2, random_gains=True)
        ls.begin()
        acc = []
        for it in range(20):
            st = ls.ctx.xsm_debug_get_state()
            drafts = None
            if it % 2 == 0:      # plant a first draft the backbone is likely to accept: its own runner-up
                drafts = st["window"][:, 1:].copy()
                for b in range(2):
                    z, _ = ls.seqs[b].forward_row(int(st["window"][b, 0]), int(st["len"][b]))
                    drafts[b, 0] = int(np.argsort(-z, kind="stable")[1])
            _, a = ls.step(drafts=drafts, margin=1e-3, **F32_TOL)
            acc.extend(a)
        assert max(acc) >= 1 and ls.excused <= 2
        ls.close()


def test_prompt_ingestion_and_eos(P):
    import oracle
    from paper_2507_23777_b200 import binding
    cfg = gpu_cfg(dtype=0, n_draft=2, sigma=0.15)
    w = inputs.make_weights(cfg, random_gains=True)
    cond = inputs.make_cond(cfg, 1)
    orc = oracle.Oracle(cfg, w, n_pages=16)
    dc = oracle.decode_config(cfg)
    prompt = [0, 5, 6, 7, 8, 9, 10, 11]
    ref = orc.new_seq(cond[0], 0).generate_plain(prompt, dc, 30)
    ctx = binding.Context(cfg, w)
    ctx.prefill(cond, prompt, binding.decode_config(cfg))
    st = ctx.xsm_debug_get_state()
    assert st["len"][0] == 7 and st["window"][0, 0] == 11
    toks, lens, _ = ctx.generate(30)
    assert np.array_equal(toks[0], ref)
    ctx.xsm_destroy()
    eos = int(ref[12])
    first = int(np.argmax(ref == eos))
    cfg_e = dict(cfg, eos_id=eos)
    ctx = binding.Context(cfg_e, w)
    ctx.prefill(cond, prompt, binding.decode_config(cfg_e))
    toks, lens, _ = ctx.generate(30)
    assert lens[0] == first + 1 and np.array_equal(toks[0, :first + 1], ref[:first + 1]) and (toks[0, first + 1:] == -1).all()
    ctx.xsm_destroy()


def test_batch_equals_independent_runs_and_k0(P):
    """A batch of sequences gives what each gives alone (own condition, own Philox stream);
    n_draft = 0 is plain decoding with SCR exactly 1."""
    from paper_2507_23777_b200 import binding
    cfg = gpu_cfg(dtype=1, n_draft=2, verify_mode=1, k_accept=2, sample_mode=1, k_sample=3, temperature=0.8, seed=3,
                  sigma=0.25)
    w = inputs.make_weights(cfg)
    cond = inputs.make_cond(cfg, 3)
    gdc = binding.decode_config(cfg)
    ctx = binding.Context(cfg, w, max_batch=3)
    ctx.prefill(cond, [0], gdc)
    toks, lens, st = ctx.generate(40)
    assert (lens == 40).all() and st.tokens == 120
    # sequence 0 alone reproduces row 0 (sequence ids are batch positions)
    ctx.prefill(cond[:1], [0], gdc)
    t0, _, _ = ctx.generate(40)
    assert np.array_equal(t0[0], toks[0])
    ctx.xsm_destroy()
    cfg0 = dict(cfg, n_draft=0)
    w0 = inputs.make_weights(cfg0)
    ctx = binding.Context(cfg0, w0)
    ctx.prefill(inputs.make_cond(cfg0, 1), [0], binding.decode_config(cfg0))
    _, lens, st = ctx.generate(25)
    assert st.steps == 25 and st.scr == 1.0 and st.accept_hist[0] == 25
    ctx.xsm_destroy()


def test_capacity_and_state_errors(P):
    from paper_2507_23777_b200 import binding
    cfg = gpu_cfg(dtype=0, n_draft=2, sigma=0.15)
    w = inputs.make_weights(cfg)
    cond = inputs.make_cond(cfg, 2)
    mc = binding.model_config(cfg, 2)
    full = binding.xsm_workspace_bytes(mc)
    page_bytes = cfg["n_layers"] * 2 * cfg["d_model"] * 32 * 4
    # room for one sequence's pages only: a batch of two is refused on the host
    ctx = binding.Context(cfg, w, max_batch=2, workspace_bytes=full - 3 * page_bytes)
    with pytest.raises(binding.XsmError) as e:
        ctx.prefill(cond, [0], binding.decode_config(cfg))
    assert e.value.status == binding.XSM_ERR_CAPACITY
    ctx.prefill(cond[:1], [0], binding.decode_config(cfg))
    ctx.generate(20)
    ctx.xsm_destroy()
    ctx = binding.Context(cfg, w, max_batch=2)
    with pytest.raises(binding.XsmError) as e:
        ctx.xsm_spec_step()
    assert e.value.status == binding.XSM_ERR_STATE
    with pytest.raises(binding.XsmError):
        ctx.prefill(cond, [0], binding.decode_config(dict(cfg, sample_mode=1, k_sample=100)))
    with pytest.raises(binding.XsmError):
        binding.Context(cfg, w, max_batch=2, workspace_bytes=4096)
    ctx.xsm_destroy()


# ---------------------------------------------------------------- long contexts, ragged batches, sampling modes on bf16


def _rank(z, r):
    """Token at rank r of logits z (larger logit first, then smaller index)."""
    return int(np.lexsort((np.arange(z.size), -z))[r])


def planted_chain(ls, b, n_good, rank=1):
    """Drafts for sequence b whose first n_good entries the backbone will accept: draft j is the token of rank `rank`
    of the oracle's backbone row j-1 given the drafts before it (the rows are run through the oracle's forward,
    which touches only cache positions the step overwrites anyway); the rest stay as they are."""
    st = ls.ctx.xsm_debug_get_state()
    n, win = int(st["len"][b]), st["window"][b].copy()
    for j in range(n_good):
        z, _ = ls.seqs[b].forward_row(int(win[j]), n + j)
        win[j + 1] = _rank(z, rank)
    return win[1:]


def test_twelve_key_splits_merge_in_two_batches(P):
    """Twelve heads of 64 leave twelve key splits per head; at a context of about 3000 tokens the last split folds in
    eleven partials, in two batches of up to eight.  The prompt is ingested by the step kernel."""
    cfg = inputs.config(1, n_layers=2, vocab=1500, n_cond=40, max_seq_len=3200)
    ls = P.LockStep(cfg, batch=1)
    prompt = [0] + [int(t) for t in np.random.default_rng(11).integers(1, cfg["vocab"], 3010)]
    st = ls.begin(prompt)
    assert st["len"][0] == len(prompt) - 1 and (-(-int(st["len"][0]) // 64) + 3) // 4 >= 12
    for _ in range(6):
        ls.step(**BF16_TOL)
    assert ls.excused <= 2
    ls.compare_cache(layers=[1], **BF16_TOL)
    ls.close()


def test_block_table_reload_after_32_pages_of_one_split(P):
    """Sixteen heads and four sequences leave two key splits per item; with 32-token pages a context of about 2400
    tokens gives each split 38 pages, so the producer fetches a second batch of block-table entries."""
    cfg = inputs.config(2, **_shape(512, 16, 32, 1024, 2, V=900, C=33, page_size=32, max_seq_len=2600))
    ls = P.LockStep(cfg, batch=4)
    prompt = [0] + [int(t) for t in np.random.default_rng(12).integers(1, cfg["vocab"], 2420)]
    st = ls.begin(prompt)
    assert (st["len"] == len(prompt) - 1).all() and -(-int(st["len"][0]) // 32) // 2 > 32
    for _ in range(6):
        ls.step(**BF16_TOL)
    assert ls.excused <= 4
    ls.compare_cache(layers=[1], **BF16_TOL)
    ls.close()


def test_context_of_twelve_thousand_tokens_at_the_width_of_configuration_2(P):
    """The regime the benchmark ends in: 16 heads of 64, nine key splits per head, 21 pages per split (a warp owns
    three of them).  One layer and a narrow feed-forward block keep the oracle's ingestion affordable."""
    cfg = inputs.config(2, n_layers=1, d_ff=1024, vocab=1500, n_cond=40, max_seq_len=12288)
    ls = P.LockStep(cfg, batch=1)
    prompt = [0] + [int(t) for t in np.random.default_rng(13).integers(1, cfg["vocab"], 12050)]
    st = ls.begin(prompt)
    assert st["len"][0] == len(prompt) - 1
    for _ in range(4):
        ls.step(**BF16_TOL)
    assert ls.excused <= 2
    n = int(ls.ctx.xsm_debug_get_state()["len"][0])
    # the cache of the last pages (appended by the steps above and by the end of the ingestion)
    k, v = ls.ctx.xsm_debug_get_kv(0, 0, n - 200, 200)
    ok = np.stack([ls.seqs[0].kv(0, 0, p) for p in range(n - 200, n)])
    ov = np.stack([ls.seqs[0].kv(0, 1, p) for p in range(n - 200, n)])
    assert P.logits_close(k, ok, **BF16_TOL).all() and P.logits_close(v, ov, **BF16_TOL).all()
    ls.close()


def test_ragged_accept_lengths_across_a_batch_of_sixteen(P):
    """Configuration 3's shape at reduced depth: sixteen meshes, top-5 acceptance, top-5 / T = 0.5 resampling.  Every
    second sequence gets drafts of which the first 1..K are the backbone's own runner-up tokens, so accept lengths
    differ across the batch and every sequence rolls back by its own amount in the shared pool."""
    cfg = inputs.config(3, n_layers=2, max_seq_len=256)
    ls = P.LockStep(cfg, batch=16)
    ls.begin()
    K, seen = cfg["n_draft"], set()
    for it in range(6):
        st = ls.ctx.xsm_debug_get_state()
        drafts = st["window"][:, 1:].copy()
        want = {}
        for b in range(0, 16, 2):
            want[b] = 1 + (b // 2 + it) % K
            drafts[b] = planted_chain(ls, b, want[b])
        _, acc = ls.step(drafts=drafts, **BF16_TOL)
        seen.update(acc)
        if ls.excused == 0:
            assert all(acc[b] >= want[b] for b in want), (acc, want)
    assert len(seen) >= 4 and ls.excused <= 6
    ls.compare_cache(layers=[1], **BF16_TOL)
    st = ls.ctx.xsm_debug_get_state()
    assert all(st["pages"][b] == -(-(st["len"][b] + K + 1) // 64) for b in range(16))
    ls.close()


@pytest.mark.parametrize("mode", ["top-5 acceptance, top-5 / T = 0.5", "threshold 0.5", "threshold 0.05"])
def test_multi_token_commits_on_a_bf16_model(P, mode):
    """Configuration 2 at reduced depth for 24 steps with planted drafts, so that several tokens are committed per
    step: with the configured rule (draft within the backbone's top 5, candidates drawn from the top 5 at T = 0.5)
    and with the paper's main rule (backbone probability of the draft above delta, Sec. 4.2)."""
    over = dict(n_layers=3, max_seq_len=512)
    if mode.startswith("threshold"):
        over.update(verify_mode=2, delta=float(mode.split()[1]))
    cfg = inputs.config(2, **over)
    ls = P.LockStep(cfg, batch=1)
    ls.begin()
    K, acc = cfg["n_draft"], []
    for it in range(24):
        # threshold: the backbone's best token (the only one that can pass 0.5); top-k: its runner-up
        drafts = planted_chain(ls, 0, it % (K + 1), rank=0 if cfg["verify_mode"] == 2 else 1)
        _, a = ls.step(drafts=np.asarray([drafts]), **BF16_TOL)
        acc.extend(a)
    assert ls.excused <= 4
    if cfg["verify_mode"] == 1:
        assert max(acc) == K and sum(acc) >= 24
    else:
        assert cfg["delta"] >= 0.5 or max(acc) >= 1, acc      # the best token of a row holds about a tenth of the mass
    ls.compare_cache(layers=[2], **BF16_TOL)
    ls.close()


def test_a_wait_that_runs_out_ends_the_kernel_cleanly_and_prefill_recovers(P):
    """A stage is launched alone whose inputs no launch has published (the out-projection of layer 0, which reads the
    attention rows), with the poll limit cut to a few thousand: every CTA gives up, finishes its ring protocol and
    leaves; the host reports XSM_ERR_TIMEOUT at the next synchronising call; the context works again after xsm_prefill.
    Nothing here faults or hangs: the wait is a bounded loop of loads that ends by counting."""
    from paper_2507_23777_b200 import binding
    cfg = gpu_cfg(dtype=1, n_draft=2, sigma=0.05)
    w = inputs.make_weights(cfg, random_gains=True)
    cond = inputs.make_cond(cfg, 1)
    dc = binding.decode_config(cfg)
    ref = binding.Context(cfg, w)
    ref.prefill(cond, [0], dc)
    want, _, _ = ref.generate(24)
    ref.xsm_destroy()
    ctx = binding.Context(cfg, w)
    ctx.prefill(cond, [0], dc)
    ctx.xsm_debug_set_wait_limits(3000, 0)
    ctx.xsm_debug_launch_stage(2)
    with pytest.raises(binding.XsmError) as e:
        ctx.xsm_debug_get_state()
    assert e.value.status == binding.XSM_ERR_TIMEOUT
    ctx.xsm_debug_set_wait_limits(0, 0)
    ctx.prefill(cond, [0], dc)
    got, lens, _ = ctx.generate(24)
    assert lens[0] == 24 and np.array_equal(got, want)
    ctx.xsm_destroy()


# ---------------------------------------------------------------- cross-attention decoding heads (Eq. 3)


@pytest.mark.parametrize("dtype,batch,phase_launch", [(0, 1, False), (1, 1, False), (1, 3, False), (0, 2, True)])
def test_cross_attention_heads_on_the_unit_model(P, dtype, batch, phase_launch):
    """head_kind 1: every head is a residual cross-attention layer with its own projections of the condition.  Logits of
    the heads, committed tokens and windows against the oracle, with scripted accept lengths."""
    cfg = gpu_cfg(dtype=dtype, n_draft=3, head_kind=1, sigma=0.15 if dtype == 0 else 0.05)
    tol = F32_TOL if dtype == 0 else BF16_TOL
    ls = P.LockStep(cfg, batch=batch, random_gains=True, phase_launch=phase_launch)
    ls.begin()
    full = []
    for b in range(batch):
        ref = ls.orc.new_seq(ls.cond[b], b).generate_plain([0], ls.odc, 60)
        full.append(np.concatenate([[0], ref]))
    rng = np.random.default_rng(1)
    for it in range(10):
        good = [int(rng.integers(0, 4)) for _ in range(batch)]
        _, acc = ls.step(drafts=scripted(ls, full, rng, good), margin=1e-3 if dtype == 0 else 1e-2, **tol)
        if ls.excused == 0:
            assert acc == good
    ls.compare_cache(**tol)
    ls.close()


def test_cross_attention_heads_at_the_width_of_configuration_2(P):
    """Configuration 2's shape at reduced depth with cross-attention heads (257 condition latents: five pages per head
    and attention head), top-5 acceptance and top-5 / T = 0.5 resampling."""
    cfg = inputs.config(2, n_layers=2, head_kind=1, max_seq_len=256)
    ls = P.LockStep(cfg, batch=1)
    ls.begin()
    for it in range(8):
        drafts = planted_chain(ls, 0, it % 3)
        ls.step(drafts=np.asarray([drafts]), **BF16_TOL)
    assert ls.excused <= 2
    ls.close()


def test_cross_attention_heads_with_split_condition_keys(P):
    """Heads of 128 and 513 condition latents (configuration 4's width at reduced depth): the condition's keys of one
    head exceed a CTA's ring, so the heads' attention is split over CTAs and merged, as the layers' is."""
    cfg = inputs.config(4, n_layers=1, d_ff=2048, n_draft=2, head_kind=1, max_seq_len=256)
    ls = P.LockStep(cfg, batch=1)
    ls.begin()
    for _ in range(3):
        ls.step(**BF16_TOL)
    ls.close()


# ---------------------------------------------------------------- probability-tree sampling (Appendix)


@pytest.mark.parametrize("dtype,K,ks", [(0, 2, 3), (1, 3, 2), (0, 4, 4)])
def test_probability_tree_sampling_lockstep(P, dtype, K, ks):
    """sample_mode 2: x_{s*} from the backbone's top-k at the configured temperature, the K drafts as one path of the
    top-k_s probability tree over the heads.  Tokens against the oracle step by step (a differing path only where the
    draw sits at an edge of the cumulative path weights or candidates nearly tie)."""
    cfg = gpu_cfg(dtype=dtype, n_draft=K, verify_mode=1, k_accept=3, sample_mode=2, k_sample=ks, temperature=0.8, seed=4,
                  sigma=0.3 if dtype == 0 else 0.1)
    ls = P.LockStep(cfg, batch=2, random_gains=True)
    ls.begin()
    paths = set()
    for it in range(24):
        ls.step(margin=1e-3 if dtype == 0 else 1e-2, **(F32_TOL if dtype == 0 else BF16_TOL))
        st = ls.ctx.xsm_debug_get_state()
        paths.add(tuple(st["window"][0, 1:].tolist()))
    assert ls.excused <= 4 and len(paths) >= 4
    ls.close()


def test_probability_tree_sampling_at_the_width_of_configuration_2(P):
    cfg = inputs.config(2, n_layers=2, sample_mode=2, k_sample=3, max_seq_len=256)
    ls = P.LockStep(cfg, batch=1)
    ls.begin()
    for _ in range(8):
        ls.step(**BF16_TOL)
    assert ls.excused <= 2
    ls.close()
