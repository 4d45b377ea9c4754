"""CPU oracle of the FlashLoop loop-r prefill step: test infrastructure, never on the product path."""
