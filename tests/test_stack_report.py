"""Host logic of the layer-stack harness: the stored-bytes accounting (no GPU needed)."""
from paper_2605_01255_b200 import inputs as I
from paper_2605_01255_b200 import stack as S


def test_stored_bytes_of_the_28_layer_stack():
    # 4 distinct inputs per decoder layer (3072, 3072, 3072, 8192), 28 layers, 16384 tokens, bf16, r = 128
    rep = S.report(I.workload("llama3b_stack28"))
    assert rep.stored_bytes_uncompressed == 28 * 16384 * (3 * 3072 + 8192) * 2 == 15_971_909_632
    assert rep.stored_bytes_compressed == 28 * 4 * 16384 * 128 * 2 == 469_762_048
    assert abs(rep.saved_bytes / rep.stored_bytes_uncompressed - 0.9706) < 1e-4
    # gradient factors against dense fp32 gradients
    per_layer_dense = 4 * (4 * 3072 * 3072 + 3 * 3072 * 8192)
    assert rep.dense_grad_bytes == 28 * per_layer_dense
    assert rep.factor_bytes == 28 * 4 * 128 * (5 * 3072 + 2 * 8192)


def test_rank_sweep_of_one_layer():
    want = {32: 4_194_304, 64: 8_388_608, 128: 16_777_216, 256: 33_554_432}
    for r, kept in want.items():
        rep = S.report(I.workload("llama3b_layer", r))
        assert rep.stored_bytes_compressed == kept
        assert rep.stored_bytes_uncompressed == 570_425_344
