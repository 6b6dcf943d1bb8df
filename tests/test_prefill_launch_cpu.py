"""Host arithmetic behind pa_prefill_split's choice of launch (no GPU): what gets split, what
the workspace allows, what a forced split length does."""
import pytest

from paper_2602_07878_b200 import api, build


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()


def shape(H, Hkv, D, nb=4096):
    return api.PaShape(H, Hkv, D, 16, nb, api.PA_BF16, Hkv * 16 * D, 16 * D, D)


def ws(sh, batch, total_q, splits):
    return api.pa_prefill_split_workspace_bytes(sh, batch, total_q, splits)


def test_recompute_chunk_of_one_long_sequence_is_split_over_the_sms():
    # 512 query tokens of a 32 K context, 32 / 8 heads: 128 row tiles for 148 SMs
    sh = shape(32, 8, 128)
    tiles, tok, splits = api.pa_prefill_select_launch(sh, 1, 512, 2048, ws(sh, 1, 512, 16))
    assert tiles == 2 and splits >= 2 and tok % 64 == 0
    assert tok * splits >= 32768 > tok * (splits - 1)         # the splits cover the context
    # 64 row groups x splits: the full-length units fill one round of the 148 SMs and the
    # shorter last split of every row group fits on the SMs they leave free
    groups = 512 // (2 * 32) * 8
    n_long, last = groups * (splits - 1), 32768 - tok * (splits - 1)
    assert n_long <= 148 and 0 < last <= tok
    if last < tok:
        per_free_sm = -(-groups // (148 - n_long))
        assert per_free_sm * last <= tok


def test_no_split_without_room_for_partial_rows_or_on_request():
    sh = shape(32, 8, 128)
    base = api.pa_prefill_workspace_bytes(1)
    assert api.pa_prefill_select_launch(sh, 1, 512, 2048, base)[1:] == (0, 1)
    assert api.pa_prefill_select_launch(sh, 1, 512, 2048, ws(sh, 1, 512, 16), -1)[1:] == (0, 1)
    # short contexts are never split: a unit must be worth its set-up
    assert api.pa_prefill_select_launch(sh, 1, 512, 32, ws(sh, 1, 512, 16))[1:] == (0, 1)
    # a call with thousands of tiles needs no split either, and takes two tiles per CTA
    assert api.pa_prefill_select_launch(sh, 1, 32768, 2048, ws(sh, 1, 32768, 4)) == (2, 0, 1)


def test_forced_split_length():
    sh = shape(32, 8, 128)
    w = ws(sh, 2, 700, 8)
    tiles, tok, splits = api.pa_prefill_select_launch(sh, 2, 700, 313, w, 1000)
    assert tok == 1024 and splits == 5 and tiles in (1, 2)   # rounded up to 64; ceil(5008 / 1024)
    with pytest.raises(api.PagedKVError) as e:
        api.pa_prefill_select_launch(sh, 2, 700, 313, w, 64)  # 79 partial rows do not fit 8
    assert e.value.code == api.ERR["WORKSPACE"]
    # a split at least as long as every context is no split
    assert api.pa_prefill_select_launch(sh, 2, 700, 313, w, 1 << 20)[1:] == (0, 1)
    with pytest.raises(api.PagedKVError) as e:
        api.pa_prefill_select_launch(sh, 2, 700, 313, api.pa_prefill_workspace_bytes(2) - 1)
    assert e.value.code == api.ERR["WORKSPACE"]


@pytest.mark.parametrize("H,Hkv,D", [(16, 8, 256), (4, 1, 256)])
def test_head_dim_256_takes_one_tile_per_cta(H, Hkv, D):
    sh = shape(H, Hkv, D)
    for total_q, blocks in [(512, 2048), (8192, 2048), (64, 8)]:
        tiles, tok, splits = api.pa_prefill_select_launch(sh, 1, total_q, blocks, ws(sh, 1, total_q, 8))
        assert tiles == 1 and splits <= 8


def test_more_sms_never_means_fewer_units():
    sh = shape(32, 8, 128)
    w = ws(sh, 1, 512, 32)
    prev = 0
    for sms in (16, 64, 148, 296):
        tiles, tok, splits = api.pa_prefill_select_launch(sh, 1, 512, 2048, w, 0, sms)
        units = -(-512 // (tiles * 32)) * 8 * splits
        assert units >= prev
        prev = units


def test_a_batch_of_short_chunks_takes_one_tile_per_cta():
    # 64 sequences of 8 query tokens each (32 / 8 heads: 32 tokens fill a 128-row tile): a
    # second tile per CTA would stay empty, so one tile it is; four sequences of 128 tokens
    # fill two tiles each
    sh = shape(32, 8, 128)
    assert api.pa_prefill_select_launch(sh, 64, 512, 32, ws(sh, 64, 512, 4))[0] == 1
    assert api.pa_prefill_select_launch(sh, 4, 512, 256, ws(sh, 4, 512, 4))[0] == 2
